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

// The same scan with four consecutive columns per thread (float4 loads and stores: a warp moves
// 512 contiguous bytes per access), used when the column count is a multiple of four.  Registers
// decide how many warps an SM holds and with them how many loads are in flight, so a thread keeps
// only the values and the local advantages of its L steps: the done flags are one bit each, and the
// running product of gamma*lambda*(1-d) is formed again, by the same multiplications in the same
// order, when the chunk's true A_in is applied.  Advantages and returns are written once and not
// read again here: streaming stores.
template <int L, int THREADS, int MINB>
__global__ void __launch_bounds__(THREADS, MINB)
gae_kernel_v4(const float *__restrict__ values, const float *__restrict__ rewards, const uint8_t *__restrict__ dones,
              float *__restrict__ adv, float *__restrict__ ret, int T, int E, int N, float gamma, float lambda) {
  static_assert(4 * L <= 32, "one done bit per step and column");
  extern __shared__ float sm[];  // [2][n_chunks][32] float4
  const int n_chunks = blockDim.y;
  float4 *sA = reinterpret_cast<float4 *>(sm), *sP = sA + n_chunks * kGaeCols;
  const size_t M = static_cast<size_t>(E) * N, M4 = M / 4;
  const size_t q = static_cast<size_t>(blockIdx.x) * kGaeCols + threadIdx.x;  // column quad
  const int chunk = threadIdx.y;
  const int t0 = chunk * L;
  const bool active = q < M4 && t0 < T;
  const int len = active ? min(L, T - t0) : 0;
  const size_t col = q * 4;
  size_t env[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) env[j] = active ? (col + j) / N : 0;
  const float gl = gamma * lambda;
  const float4 *v4 = reinterpret_cast<const float4 *>(values), *r4 = reinterpret_cast<const float4 *>(rewards);

  float4 v[L], r[L];
  uint32_t alive = 0;  // bit 4 i + j: column j is not done at step i
#pragma unroll
  for (int i = 0; i < L; ++i) {
    if (i < len) {
      const size_t t = static_cast<size_t>(t0 + i);
      v[i] = __ldg(v4 + t * M4 + q);
      r[i] = __ldg(r4 + t * M4 + q);
      const uint8_t *d = dones + t * E;
#pragma unroll
      for (int j = 0; j < 4; ++j) alive |= (__ldg(d + env[j]) ? 0u : 1u) << (4 * i + j);
    }
  }
  const float4 v_after = active ? __ldg(v4 + static_cast<size_t>(t0 + len) * M4 + q) : make_float4(0.f, 0.f, 0.f, 0.f);
  auto keep = [&](int i) {
    return make_float4(static_cast<float>((alive >> (4 * i)) & 1u), static_cast<float>((alive >> (4 * i + 1)) & 1u),
                       static_cast<float>((alive >> (4 * i + 2)) & 1u), static_cast<float>((alive >> (4 * i + 3)) & 1u));
  };
  // in place: r becomes the local advantage (A_in = 0)
  float4 a_run = make_float4(0.f, 0.f, 0.f, 0.f), p_run = make_float4(1.f, 1.f, 1.f, 1.f);
#pragma unroll
  for (int i = L - 1; i >= 0; --i) {
    if (i < len) {
      const float4 vn = (i == len - 1 || i == L - 1) ? v_after : v[i + 1 < L ? i + 1 : i];
      const float4 ci = keep(i);
      a_run.x = (r[i].x + gamma * vn.x * ci.x - v[i].x) + gl * ci.x * a_run.x;
      a_run.y = (r[i].y + gamma * vn.y * ci.y - v[i].y) + gl * ci.y * a_run.y;
      a_run.z = (r[i].z + gamma * vn.z * ci.z - v[i].z) + gl * ci.z * a_run.z;
      a_run.w = (r[i].w + gamma * vn.w * ci.w - v[i].w) + gl * ci.w * a_run.w;
      p_run.x = gl * ci.x * p_run.x; p_run.y = gl * ci.y * p_run.y;
      p_run.z = gl * ci.z * p_run.z; p_run.w = gl * ci.w * p_run.w;
      r[i] = a_run;
    }
  }
  sA[chunk * kGaeCols + threadIdx.x] = a_run;
  sP[chunk * kGaeCols + threadIdx.x] = p_run;
  __syncthreads();
  if (!active) return;
  float4 a_in = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int k = n_chunks - 1; k > chunk; --k) {
    const float4 a = sA[k * kGaeCols + threadIdx.x], p = sP[k * kGaeCols + threadIdx.x];
    a_in = make_float4(a.x + p.x * a_in.x, a.y + p.y * a_in.y, a.z + p.z * a_in.z, a.w + p.w * a_in.w);
  }
  float4 *adv4 = reinterpret_cast<float4 *>(adv), *ret4 = reinterpret_cast<float4 *>(ret);
  float4 p = make_float4(1.f, 1.f, 1.f, 1.f);
#pragma unroll
  for (int i = L - 1; i >= 0; --i) {
    if (i < len) {
      const size_t t = static_cast<size_t>(t0 + i);
      const float4 ci = keep(i);
      p.x = gl * ci.x * p.x; p.y = gl * ci.y * p.y; p.z = gl * ci.z * p.z; p.w = gl * ci.w * p.w;
      const float4 a = make_float4(r[i].x + p.x * a_in.x, r[i].y + p.y * a_in.y, r[i].z + p.z * a_in.z, r[i].w + p.w * a_in.w);
      __stcs(adv4 + t * M4 + q, a);
      __stcs(ret4 + t * M4 + q, make_float4(a.x + v[i].x, a.y + v[i].y, a.z + v[i].z, a.w + v[i].w));
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
  // the float4 variant pays off once there are enough columns to fill the GPU with its larger blocks
  const bool vec = M % 4 == 0 && M >= 16384 && reinterpret_cast<uintptr_t>(b.values) % 16 == 0 && reinterpret_cast<uintptr_t>(b.rewards) % 16 == 0 &&
                   reinterpret_cast<uintptr_t>(b.adv) % 16 == 0 && reinterpret_cast<uintptr_t>(b.ret) % 16 == 0;
  const unsigned blocks4 = static_cast<unsigned>((M / 4 + kGaeCols - 1) / kGaeCols);
  auto go4 = [&](auto kern, int L) {
    const int n_chunks = (T + L - 1) / L;
    kern<<<blocks4, dim3(kGaeCols, n_chunks), 2 * static_cast<size_t>(n_chunks) * kGaeCols * sizeof(float4), h->stream>>>(
        b.values, b.rewards, b.dones, b.adv, b.ret, T, E, N, gamma, lambda);
  };
  // chunks of four steps: 16 or 32 warps per block, few registers per thread, so that an SM holds 32 warps
  // with eight 16-byte loads each in flight (measured against chunks of eight: 74 -> 63 us on 64 x 262144)
  if (vec && T <= 4 * 16) {
    go4(gae_kernel_v4<4, 512, 2>, 4);
  } else if (vec && T <= 4 * 32) {
    go4(gae_kernel_v4<4, 1024, 1>, 4);
  } else if (T <= 8 * 32) go(gae_kernel<8>, 8);
  else if (T <= 16 * 32) go(gae_kernel<16>, 16);
  else if (T <= 32 * 32) go(gae_kernel<32>, 32);
  else return cudaErrorInvalidValue;
  h->launches += 1;
  return cudaGetLastError();
}

}  // namespace mava
