// Rollout with the recurrent policy, fp32 SIMT path (the validation path of this net): the loop of rollout_simt.cu
// with a gated recurrent unit in place of the second hidden layer.  One CTA owns a tile of environments for all T
// steps; environment states, the observation tile, the embedding, the six gate pre-activations and the agents' hidden
// vectors stay in shared memory.  The hidden vectors come from and go back to a per-handle array [E][N][H]; a step
// that ends an episode zeroes the vectors of that environment's agents.  The bootstrap step (t == T) updates a copy.
#include "common.cuh"
#include "env.cuh"
#include "layout.h"
#include "simt_dense.cuh"

namespace mava {
namespace {

struct RecWeights {
  const float *W1t, *b1;           // [D][H]
  const float *Wit[3], *bi[3];     // input part of gate g: [H][H] transposed, bias [H]
  const float *Wht[3], *bh[3];     // hidden part
  const float *Wa, *ba, *Wv, *bv;  // heads, row-major
};

template <int N, int F, int H>
struct RecSmem {
  static constexpr int D = kObsFixed + N;
  static constexpr int EPT = kSimtRows / N;
  static constexpr int HS = H + 1;
  EnvRec st[EPT];
  alignas(16) float obs[kSimtRows * D];
  float emb[kSimtRows * HS];
  float gi[3][kSimtRows * HS], gh[3][kSimtRows * HS];
  float hid[kSimtRows * HS];   // carried
  float hnew[kSimtRows * HS];  // this step's new hidden vectors (the heads read these)
  float logits[kSimtRows * 8];
  float value[kSimtRows];
  int act[kSimtRows];
  uint8_t new_r[kSimtRows], new_c[kSimtRows], collected[EPT * F], done[EPT];
};

__device__ __forceinline__ float sigmoidf_(float v) { return 1.0f / (1.0f + expf(-v)); }

template <int N, int F, int H>
__global__ void __launch_bounds__(kSimtThreads)
rollout_rec_simt_kernel(RolloutArgs a, RecWeights w, float *__restrict__ hidden) {
  using S = RecSmem<N, F, H>;
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
  for (int i = tid; i < kSimtRows * H; i += kSimtThreads) {
    const int row = i / H, j = i - row * H;
    sm.hid[row * HS + j] = row < n_rows ? hidden[(static_cast<size_t>(e0) * N + row) * H + j] : 0.0f;
  }
  __syncthreads();

  for (int t = 0; t <= a.T; ++t) {
    const bool last = t == a.T;
    const size_t row0 = static_cast<size_t>(t) * M + static_cast<size_t>(e0) * N;
    auto sink = [&](int row, int j, float v) { sm.obs[row * D + j] = v; };
    observe_fill<N>(sm.st, a.env, n_rows, tid, kSimtThreads, sink);
    __syncthreads();
    observe_scatter<N, F>(sm.st, n_rows, tid, kSimtThreads, sink);
    __syncthreads();
    if (!last) {
      float *dst = a.buf.obs + row0 * D;
      for (int i = tid; i < n_rows * D; i += kSimtThreads) dst[i] = sm.obs[i];
    }
    dense_tile<D, H, kSimtRows, true>(sm.obs, D, w.W1t, w.b1, sm.emb, HS, tid);
    __syncthreads();
#pragma unroll
    for (int g = 0; g < 3; ++g) {
      dense_tile<H, H, kSimtRows, false>(sm.emb, HS, w.Wit[g], w.bi[g], sm.gi[g], HS, tid);
      dense_tile<H, H, kSimtRows, false>(sm.hid, HS, w.Wht[g], w.bh[g], sm.gh[g], HS, tid);
    }
    __syncthreads();
    for (int i = tid; i < kSimtRows * H; i += kSimtThreads) {
      const int row = i / H, j = i - row * H, k = row * HS + j;
      const float r = sigmoidf_(sm.gi[0][k] + sm.gh[0][k]);
      const float z = sigmoidf_(sm.gi[1][k] + sm.gh[1][k]);
      const float c = tanhf(sm.gi[2][k] + r * sm.gh[2][k]);
      sm.hnew[k] = (1.0f - z) * c + z * sm.hid[k];
    }
    __syncthreads();
    if (tid < kSimtRows * (kActions + 1)) {  // heads: one thread per (row, output)
      const int row = tid / (kActions + 1), o = tid - row * (kActions + 1);
      const float *wrow = (o < kActions) ? w.Wa + o * H : w.Wv;
      float acc = 0.0f;
      for (int k = 0; k < H; ++k) acc = fmaf(sm.hnew[row * HS + k], __ldg(wrow + k), acc);
      if (o < kActions) sm.logits[row * 8 + o] = acc + __ldg(w.ba + o);
      else sm.value[row] = acc + __ldg(w.bv);
    }
    __syncthreads();
    if (tid < n_rows) {
      a.buf.values[row0 + tid] = sm.value[tid];
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
        float la = l[0];
#pragma unroll
        for (int k = 1; k < kActions; ++k) la = (action == k) ? l[k] : la;
        sm.act[tid] = action;
        a.buf.actions[row0 + tid] = action;
        a.buf.logp[row0 + tid] = la - m - logf(sum);
        if (a.write_logits) {
#pragma unroll
          for (int k = 0; k < kActions; ++k) a.buf.logits[(row0 + tid) * kActions + k] = l[k];
        }
      }
    }
    __syncthreads();
    if (last) break;

    step_decide<N, F>(sm.st, a.env, sm.act, n_env, sm.new_r, sm.new_c, sm.collected, tid, kSimtThreads);
    __syncthreads();
    if (tid < n_env) {
      float reward;
      bool done;
      step_apply<N, F>(sm.st[tid], a.env, static_cast<uint32_t>(a.env.first_env + e0 + tid), sm.new_r, sm.new_c,
                       sm.collected, tid, reward, done);
      for (int n = 0; n < N; ++n) a.buf.rewards[row0 + tid * N + n] = reward;
      a.buf.dones[static_cast<size_t>(t) * a.env.n_envs + e0 + tid] = done ? 1 : 0;
      sm.done[tid] = done ? 1 : 0;
    }
    __syncthreads();
    // the new hidden vectors become the carried ones; a finished episode leaves no memory behind
    for (int i = tid; i < kSimtRows * H; i += kSimtThreads) {
      const int row = i / H, j = i - row * H, k = row * HS + j;
      sm.hid[k] = (row < n_rows && sm.done[row / N]) ? 0.0f : sm.hnew[k];
    }
    __syncthreads();
  }
  for (int i = tid; i < n_rows * H; i += kSimtThreads) {
    const int row = i / H, j = i - row * H;
    hidden[(static_cast<size_t>(e0) * N + row) * H + j] = sm.hid[row * HS + j];
  }
  for (int i = tid; i < n_env * static_cast<int>(sizeof(EnvRec) / 4); i += kSimtThreads)
    reinterpret_cast<uint32_t *>(a.state + e0)[i] = reinterpret_cast<const uint32_t *>(sm.st)[i];
}

// [out][in] matrices transposed to [in][out] (the cell's, one gate block at a time); the rest copied.
__global__ void prep_rec_simt_kernel(const float *__restrict__ src, float *__restrict__ dst, ParamLayout in, ParamLayout out, int D, int H) {
  const size_t tid = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x;
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  auto transpose = [&](size_t s, size_t d, int rows_out, int cols_in) {
    const size_t n = static_cast<size_t>(rows_out) * cols_in;
    for (size_t i = tid; i < n; i += stride) {
      const size_t k = i / rows_out, o = i - k * rows_out;
      dst[d + i] = src[s + o * cols_in + k];
    }
  };
  auto copy = [&](size_t s, size_t d, size_t n) {
    for (size_t i = tid; i < n; i += stride) dst[d + i] = src[s + i];
  };
  transpose(in.W1, out.W1, H, D); copy(in.b1, out.b1, H);
  for (int g = 0; g < 3; ++g) {
    transpose(in.Wih + static_cast<size_t>(g) * H * H, out.Wih + static_cast<size_t>(g) * H * H, H, H);
    transpose(in.Whh + static_cast<size_t>(g) * H * H, out.Whh + static_cast<size_t>(g) * H * H, H, H);
  }
  copy(in.bih, out.bih, 3 * static_cast<size_t>(H)); copy(in.bhh, out.bhh, 3 * static_cast<size_t>(H));
  copy(in.Wa, out.Wa, static_cast<size_t>(kActions) * H); copy(in.ba, out.ba, kActions);
  copy(in.Wv, out.Wv, H); copy(in.bv, out.bv, 1);
}

template <int N, int F, int H>
cudaError_t launch_rec_simt_variant(mava_rollout *h, const RolloutArgs &args, const RecWeights &w) {
  using S = RecSmem<N, F, H>;
  auto kern = rollout_rec_simt_kernel<N, F, H>;
  const size_t smem = sizeof(S);
  cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (err != cudaSuccess) return err;
  const int tiles = (h->cfg.n_envs + S::EPT - 1) / S::EPT;
  kern<<<tiles, kSimtThreads, smem, h->stream>>>(args, w, h->d_hidden);
  h->launches += 1;
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_rollout_rec_simt(mava_rollout *h, const float *params_dev, const RolloutArgs &args) {
  const int H = h->cfg.hidden;
  const ParamLayout in = param_layout(h->cfg, h->D, 1), L = param_layout(h->cfg, h->D, 4);
  prep_rec_simt_kernel<<<148, 256, 0, h->stream>>>(params_dev, h->d_wsimt, in, L, h->D, H);
  h->launches += 1;
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  const float *base = h->d_wsimt;
  RecWeights w{};
  w.W1t = base + L.W1; w.b1 = base + L.b1;
  for (int g = 0; g < 3; ++g) {
    w.Wit[g] = base + L.Wih + static_cast<size_t>(g) * H * H; w.bi[g] = base + L.bih + static_cast<size_t>(g) * H;
    w.Wht[g] = base + L.Whh + static_cast<size_t>(g) * H * H; w.bh[g] = base + L.bhh + static_cast<size_t>(g) * H;
  }
  w.Wa = base + L.Wa; w.ba = base + L.ba; w.Wv = base + L.Wv; w.bv = base + L.bv;
  switch (h->variant) {
    case 5: return launch_rec_simt_variant<2, 2, 64>(h, args, w);
    case 6: return launch_rec_simt_variant<3, 3, 64>(h, args, w);
    default: return cudaErrorNotSupported;
  }
}

}  // namespace mava
