// Generalised advantage estimation as a chunked reverse scan.
//
// A_t = delta_t + c_t * A_{t+1} with c_t = gamma*lambda*(1-d_t) is an affine recurrence, so a
// column's T steps are cut into chunks of L steps that are scanned independently (local result
// for A_in = 0 plus the running product of c), the chunk summaries are chained through shared
// memory, and every element is fixed up with its chunk's true A_in.  A warp covers 32 consecutive
// (env, agent) columns at one time step, so every load and store is a full 128-byte line of the
// time-major arrays; all loads of a thread are independent of the recurrence.
#include "common.cuh"

namespace mava {
namespace {

constexpr int kGaeCols = 32;

template <int L>
__global__ void gae_kernel(const float *__restrict__ values, const float *__restrict__ rewards,
                           const uint8_t *__restrict__ dones, float *__restrict__ adv,
                           float *__restrict__ ret, int T, int E, int N, float gamma, float lambda) {
  extern __shared__ float sm[];  // [2][n_chunks][32]
  const int n_chunks = blockDim.y;
  float *sA = sm, *sP = sm + n_chunks * kGaeCols;
  const size_t M = static_cast<size_t>(E) * N;
  const size_t col = static_cast<size_t>(blockIdx.x) * kGaeCols + threadIdx.x;
  const int chunk = threadIdx.y;
  const int t0 = chunk * L;
  const bool active = col < M && t0 < T;
  const int len = active ? min(L, T - t0) : 0;
  const size_t e = active ? col / N : 0;
  const float gl = gamma * lambda;

  float v[L], r[L], c[L];
#pragma unroll
  for (int i = 0; i < L; ++i) {
    if (i < len) {
      const size_t t = static_cast<size_t>(t0 + i);
      v[i] = values[t * M + col];
      r[i] = rewards[t * M + col];
      c[i] = dones[t * E + e] ? 0.0f : 1.0f;
    }
  }
  // V at the step after the chunk
  float v_after = active ? values[static_cast<size_t>(t0 + len) * M + col] : 0.0f;

  float a_loc[L], p[L];
  float a_run = 0.0f, p_run = 1.0f;
#pragma unroll
  for (int i = L - 1; i >= 0; --i) {
    if (i < len) {
      const float v_next = (i == len - 1 || i == L - 1) ? v_after : v[i + 1 < L ? i + 1 : i];
      const float delta = r[i] + gamma * v_next * c[i] - v[i];
      a_run = delta + gl * c[i] * a_run;
      p_run = gl * c[i] * p_run;
      a_loc[i] = a_run;
      p[i] = p_run;
    }
  }
  sA[chunk * kGaeCols + threadIdx.x] = a_run;  // value at the chunk's first step (A_in = 0)
  sP[chunk * kGaeCols + threadIdx.x] = p_run;
  __syncthreads();
  if (!active) return;
  float a_in = 0.0f;  // A at the first step of the next chunk
  for (int k = n_chunks - 1; k > chunk; --k)
    a_in = sA[k * kGaeCols + threadIdx.x] + sP[k * kGaeCols + threadIdx.x] * a_in;
#pragma unroll
  for (int i = 0; i < L; ++i) {
    if (i < len) {
      const size_t t = static_cast<size_t>(t0 + i);
      const float a = a_loc[i] + p[i] * a_in;
      adv[t * M + col] = a;
      ret[t * M + col] = a + v[i];
    }
  }
}

}  // namespace

cudaError_t launch_gae(mava_rollout *h, float gamma, float lambda) {
  const int T = h->last_T, E = h->cfg.n_envs, N = h->cfg.n_agents;
  const size_t M = static_cast<size_t>(E) * N;
  const unsigned blocks = static_cast<unsigned>((M + kGaeCols - 1) / kGaeCols);
  const mava_buffers_t &b = h->buf;
  auto go = [&](auto kern, int L) {
    const int n_chunks = (T + L - 1) / L;
    const size_t smem = 2 * static_cast<size_t>(n_chunks) * kGaeCols * sizeof(float);
    kern<<<blocks, dim3(kGaeCols, n_chunks), smem, h->stream>>>(b.values, b.rewards, b.dones, b.adv, b.ret, T, E, N,
                                                                gamma, lambda);
  };
  if (T <= 8 * 32) go(gae_kernel<8>, 8);
  else if (T <= 16 * 32) go(gae_kernel<16>, 16);
  else if (T <= 32 * 32) go(gae_kernel<32>, 32);
  else return cudaErrorInvalidValue;
  h->launches += 1;
  return cudaGetLastError();
}

}  // namespace mava
