// Generalised advantage estimation as a chunked reverse scan.
//
// A_t = delta_t + c_t * A_{t+1} with c_t = gamma*lambda*(1-d_t) is an affine recurrence, so a
// column's T steps are cut into chunks of L steps that are scanned independently (local result
// for A_in = 0 plus the running product of c), the chunk summaries are chained through shared
// memory, and every element is fixed up with its chunk's true A_in.  A warp covers 32 consecutive
// (env, agent) columns at one time step, so every load and store is a full 128-byte line of the
// time-major arrays; all loads of a thread are independent of the recurrence.
#include "common.cuh"
#include "tc_common.cuh"
#include "tmap.cuh"

namespace mava {
namespace {

constexpr int kGaeCols = 32;

__device__ __forceinline__ float4 lds_f32x4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t lds_u8(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void mbar_arrive_local(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

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

// The scan as a persistent kernel fed by the tiled copy engine.  A CTA per SM walks over column tiles of C
// columns; one thread asks for a tile's values [T+1][C] and rewards [T][C] with tensor-map copies into a ring
// of three shared-memory stages, so two tiles (about 130 KB per SM) are always on their way while a third is
// scanned, and neither registers nor warps are tied up by loads in flight.  The done flags of the tile's
// environments come the same way (a byte box of W columns starting on a 16-byte boundary): fetched by plain
// loads one tile ahead they made every tile wait out a memory latency, which under a saturated memory system
// is longer than a tile takes.  Thread (chunk, quad) reads its four steps of four columns and their done
// bytes from the stage, lets go of the stage, scans, chains the chunks through shared memory and writes
// advantages and returns with streaming 16-byte stores.  The done flag selects the factor (gamma or 0,
// gamma lambda or 0) instead of multiplying it in.  Every mbarrier wait is bounded.
constexpr int kGaeStages = 3, kGaeL = 4;

template <int MAXT>
__global__ void __launch_bounds__(MAXT, 1)
gae_tma_kernel(const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_r,
               const __grid_constant__ CUtensorMap map_d, float *__restrict__ adv, float *__restrict__ ret, int T, int E, int N, int C,
               int W, int n_tiles, float gamma, float lambda, int *status, int debug_expire) {
  constexpr int L = kGaeL, S = kGaeStages;
  extern __shared__ __align__(128) unsigned char smem[];
  const int QW = C / 4;  // column quads per tile row
  const int n_chunks = (T + L - 1) / L;
  const int tid = threadIdx.x, q = tid % QW, chunk = tid / QW;
  const int t0 = chunk * L;
  const bool worker = chunk < n_chunks;  // the block is rounded up to whole warps
  const int len = worker ? min(L, T - t0) : 0;
  const uint32_t d_off = static_cast<uint32_t>(2 * T + 1) * C * 4;  // values, rewards, then the done bytes [T][W]
  const uint32_t stage_bytes = d_off + static_cast<uint32_t>(T) * W;
  const uint32_t stage_stride = (stage_bytes + 127u) & ~127u;
  const uint32_t smem0 = smem_u32(smem);
  float4 *sA = reinterpret_cast<float4 *>(smem + S * stage_stride), *sP = sA + n_chunks * QW;
  uint64_t *bars = reinterpret_cast<uint64_t *>(sP + n_chunks * QW);
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8u * S;
  const int n_warps = (blockDim.x + 31) / 32;
  if (tid == 0) {
    for (int i = 0; i < S; ++i) {
      mbar_init(full0 + 8u * i, 1);
      mbar_init(empty0 + 8u * i, n_warps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const int my_tiles = (n_tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
  // first column of this CTA's i-th tile (column indices fit 32 bits: the launcher checks)
  auto tile_col = [&](int i) { return (static_cast<uint32_t>(blockIdx.x) + static_cast<uint32_t>(i) * gridDim.x) * static_cast<uint32_t>(C); };
  auto request = [&](int i) {  // one thread: tile i of this CTA into stage i % S
    const uint32_t dst = smem0 + static_cast<uint32_t>(i % S) * stage_stride, bar = full0 + 8u * (i % S);
    const uint32_t x = tile_col(i);
    mbar_expect_tx(bar, stage_bytes);
    tma_load_2d(dst, &map_v, static_cast<int>(x), 0, bar);
    tma_load_2d(dst + static_cast<uint32_t>(T + 1) * C * 4, &map_r, static_cast<int>(x), 0, bar);
    // from the 16-byte boundary at or below the tile's first environment
    tma_load_2d(dst + d_off, &map_d, static_cast<int>((x / static_cast<uint32_t>(N)) & ~15u), 0, bar);
  };
  const size_t M = static_cast<size_t>(E) * N;
  const float gl = gamma * lambda;

  bool timed_out = false;
  int issued = 0;
  if (tid == 0)
    for (; issued < S - 1 && issued < my_tiles; ++issued) request(issued);
#pragma unroll 1
  for (int i = 0; i < my_tiles; ++i) {
    const int s = i % S;
    if (tid == 0 && issued < my_tiles) {
      // the stage of tile i - 1 is the one tile i + S - 1 goes into: every warp let go of it an iteration ago
      if (i > 0) timed_out |= !mbar_wait(empty0 + 8u * ((i - 1) % S), ((i - 1) / S) & 1);
      if (!timed_out) { request(issued); ++issued; }
    }
    timed_out |= !mbar_wait(full0 + 8u * s, (i / S) & 1);
    // self-test of the give-up path: block 0, at its last tile (every copy it asked for has landed by now), waits
    // briefly for the phase of this stage that no further copy will complete
    if (debug_expire && blockIdx.x == 0 && tid == 0 && i == my_tiles - 1)
      timed_out |= !mbar_wait(full0 + 8u * s, ((i / S) & 1) ^ 1, 1u << 12);
    if (__syncthreads_or(timed_out)) { timed_out = true; break; }
    const uint32_t vbase = smem0 + static_cast<uint32_t>(s) * stage_stride, rbase = vbase + static_cast<uint32_t>(T + 1) * C * 4;
    // bit 4 k + j: column j of this thread's quad is not done at step t0 + k.  One division per tile; the quad's
    // other columns follow by counting.
    uint32_t alive = 0;
    {
      const uint32_t col0 = tile_col(i), colq = col0 + 4u * q;
      const uint32_t env0 = colq / static_cast<uint32_t>(N), x0 = (col0 / static_cast<uint32_t>(N)) & ~15u;
      uint32_t rem = colq - env0 * static_cast<uint32_t>(N), e = env0 - x0;
      const uint32_t dbase = vbase + d_off + static_cast<uint32_t>(t0 * W);
      uint32_t done[L];
#pragma unroll
      for (int k = 0; k < L; ++k) done[k] = k < len ? lds_u8(dbase + static_cast<uint32_t>(k * W) + e) : 0u;
#pragma unroll
      for (int k = 0; k < L; ++k) alive |= (done[k] ? 0u : 1u) << (4 * k);
#pragma unroll
      for (int j = 1; j < 4; ++j) {
        if (++rem == static_cast<uint32_t>(N)) {  // column j opens the next environment
          rem = 0;
          ++e;
#pragma unroll
          for (int k = 0; k < L; ++k) done[k] = k < len ? lds_u8(dbase + static_cast<uint32_t>(k * W) + e) : 0u;
        }
#pragma unroll
        for (int k = 0; k < L; ++k) alive |= (done[k] ? 0u : 1u) << (4 * k + j);
      }
    }
    float4 v[L], r[L], v_after = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int k = 0; k < L; ++k) {
      if (k < len) {
        v[k] = lds_f32x4(vbase + static_cast<uint32_t>((t0 + k) * C + 4 * q) * 4);
        r[k] = lds_f32x4(rbase + static_cast<uint32_t>((t0 + k) * C + 4 * q) * 4);
      }
    }
    if (len > 0) v_after = lds_f32x4(vbase + static_cast<uint32_t>((t0 + len) * C + 4 * q) * 4);
    // gamma (1 - d) and gamma lambda (1 - d) of column j at step k, picked by the done bit
    auto gam = [&](int k, int j) { return (alive >> (4 * k + j)) & 1u ? gamma : 0.0f; };
    auto dec = [&](int k, int j) { return (alive >> (4 * k + j)) & 1u ? gl : 0.0f; };
    float4 a_run = make_float4(0.f, 0.f, 0.f, 0.f), p_run = make_float4(1.f, 1.f, 1.f, 1.f);
#pragma unroll
    for (int k = L - 1; k >= 0; --k) {
      if (k < len) {
        const float4 vn = (k == len - 1 || k == L - 1) ? v_after : v[k + 1 < L ? k + 1 : k];
        a_run.x = fmaf(dec(k, 0), a_run.x, fmaf(gam(k, 0), vn.x, r[k].x - v[k].x));
        a_run.y = fmaf(dec(k, 1), a_run.y, fmaf(gam(k, 1), vn.y, r[k].y - v[k].y));
        a_run.z = fmaf(dec(k, 2), a_run.z, fmaf(gam(k, 2), vn.z, r[k].z - v[k].z));
        a_run.w = fmaf(dec(k, 3), a_run.w, fmaf(gam(k, 3), vn.w, r[k].w - v[k].w));
        p_run.x *= dec(k, 0); p_run.y *= dec(k, 1); p_run.z *= dec(k, 2); p_run.w *= dec(k, 3);
        r[k] = a_run;  // in place: r becomes the local advantage (A_in = 0)
      }
    }
    if (worker) {
      sA[chunk * QW + q] = a_run;  // after the scan, which consumed every value read from the stage
      sP[chunk * QW + q] = p_run;
    }
    __syncwarp();
    if ((tid & 31) == 0) mbar_arrive_local(empty0 + 8u * s);
    __syncthreads();
    float4 a_in = make_float4(0.f, 0.f, 0.f, 0.f);
    if (worker)
      for (int k = n_chunks - 1; k > chunk; --k) {
        const float4 a = sA[k * QW + q], p = sP[k * QW + q];
        a_in = make_float4(fmaf(p.x, a_in.x, a.x), fmaf(p.y, a_in.y, a.y), fmaf(p.z, a_in.z, a.z), fmaf(p.w, a_in.w, a.w));
      }
    __syncthreads();  // the summaries may be overwritten by the next tile
    const size_t col = static_cast<size_t>(tile_col(i)) + 4u * q;
    if (len > 0 && col < M) {
      float4 *adv4 = reinterpret_cast<float4 *>(adv + col), *ret4 = reinterpret_cast<float4 *>(ret + col);
      const size_t M4 = M / 4;
      float4 p = make_float4(1.f, 1.f, 1.f, 1.f);
#pragma unroll
      for (int k = L - 1; k >= 0; --k) {
        if (k < len) {
          const size_t t = static_cast<size_t>(t0 + k);
          p.x *= dec(k, 0); p.y *= dec(k, 1); p.z *= dec(k, 2); p.w *= dec(k, 3);
          const float4 a = make_float4(fmaf(p.x, a_in.x, r[k].x), fmaf(p.y, a_in.y, r[k].y), fmaf(p.z, a_in.z, r[k].z),
                                       fmaf(p.w, a_in.w, r[k].w));
          __stcs(adv4 + t * M4, a);
          __stcs(ret4 + t * M4, make_float4(a.x + v[k].x, a.y + v[k].y, a.z + v[k].z, a.w + v[k].w));
        }
      }
    }
  }
  if (timed_out) {
    if (tid == 0) {
      atomicExch(status, kStatusTimeout);
      // let the copies still in flight land before the block goes away
      for (int j = issued > S ? issued - S : 0; j < issued; ++j) mbar_wait(full0 + 8u * (j % S), (j / S) & 1);
    }
    __syncthreads();
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
  // The persistent copy-engine kernel where there is enough work for it and the tile geometry fits.
  if (vec && T >= 16 && T <= 255 && M < (1ull << 31) && E % 16 == 0 && reinterpret_cast<uintptr_t>(b.dones) % 16 == 0) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->device) != cudaSuccess) return cudaErrorUnknown;
    // columns per tile: as wide as three stages of (2 T + 1) rows allow, but at least four tiles per SM
    int C = 128, W = 0, threads = 0;
    size_t smem = 0;
    const int n_chunks = (T + kGaeL - 1) / kGaeL;
    for (;; C /= 2) {
      W = (15 + (C - 1) / N + 2 + 15) / 16 * 16;  // environments under C columns from any start, plus the way back to the boundary
      const size_t stage = (static_cast<size_t>(2 * T + 1) * C * 4 + static_cast<size_t>(T) * W + 127) / 128 * 128;
      smem = kGaeStages * stage + 2 * static_cast<size_t>(n_chunks) * (C / 4) * sizeof(float4) + 2 * kGaeStages * 8;
      threads = ((C / 4) * n_chunks + 31) / 32 * 32;
      if (C == 32 || (smem <= 232000 && threads <= 1024 && M / C >= static_cast<size_t>(4 * sms))) break;
    }
    CUtensorMap map_v, map_r, map_d;
    if (threads <= 1024 && smem <= 232000 && W <= 256 &&
        encode_f32_map(&map_v, b.values, M, static_cast<unsigned long long>(T) + 1, C, T + 1, CU_TENSOR_MAP_SWIZZLE_NONE) &&
        encode_f32_map(&map_r, b.rewards, M, T, C, T, CU_TENSOR_MAP_SWIZZLE_NONE) &&
        encode_map_2d(&map_d, b.dones, true, E, T, W, T, CU_TENSOR_MAP_SWIZZLE_NONE)) {
      const int n_tiles = static_cast<int>((M + C - 1) / C);
      const int expire = (h->expire_next & MAVA_EXPIRE_GAE) ? 1 : 0;
      h->expire_next &= ~MAVA_EXPIRE_GAE;
      auto run = [&](auto kern) {
        cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (err != cudaSuccess) return err;
        kern<<<n_tiles < sms ? n_tiles : sms, threads, smem, h->stream>>>(map_v, map_r, map_d, b.adv, b.ret, T, E, N, C, W, n_tiles,
                                                                          gamma, lambda, h->d_status, expire);
        h->launches += 1;
        return cudaGetLastError();
      };
      return threads <= 512 ? run(gae_tma_kernel<512>) : run(gae_tma_kernel<1024>);
    }
  }
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
