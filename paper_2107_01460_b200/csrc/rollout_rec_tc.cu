// Rollout with the recurrent policy on the tensor cores (sm_100a, tcgen05; H = 64): the fused loop of rollout_tc.cu
// with a gated recurrent unit between the embedding and the heads.  One persistent CTA per SM, 128 threads; thread r
// owns agent row r of its tile (= tensor-memory lane r) and keeps the environment in registers (env.cuh).  Per step:
//   1. non-zero observation entries into a zeroed bf16 A tile and a zeroed fp32 block (the block leaves as one bulk
//      copy into the time-major obs array);
//   2. MMAs: embedding pre-activation x . W1^T, and straight away the hidden part of the three gates from the carried
//      hidden tile (h . Whr^T, h . Whz^T into the r|z accumulator, h . Whn^T into its own);
//   3. epilogue: e = relu(. + b1) as a bf16 tile; MMAs: the input part e . Wir^T, e . Wiz^T on top of the r|z
//      accumulator, e . Win^T into its own;
//   4. gate epilogue in fp32 (thread = row): r, z, n, h' = (1 - z) n + z h; h' rounded to bf16 replaces the row of the
//      hidden tile (the carried state is that bf16 number, as in the oracle's bf16-operand mode);
//   5. heads MMA on the new hidden tile; sampler; warp-level transition; a finished episode zeroes its agents' rows
//      of the hidden tile.
// The bootstrap step (t == T) writes h' into the embedding tile instead, so the carried state is not advanced.
// The hidden vectors live in a per-handle fp32 array between runs.  Every mbarrier wait is bounded.
#include <cuda_bf16.h>

#include "common.cuh"
#include "env.cuh"
#include "layout.h"
#include "tc_common.cuh"

namespace mava {
namespace {

constexpr int kRH = 64;    // hidden width
constexpr int kRK1 = 80;   // input width, padded (D = 79, 80)

// weight image
constexpr uint32_t kW1 = 0, kWih = kW1 + kRH * kRK1 * 2, kWhh = kWih + 3 * kRH * kRH * 2, kWh = kWhh + 3 * kRH * kRH * 2;
constexpr uint32_t kB1 = kWh + kHeadRows * kRH * 2, kBrz = kB1 + kRH * 4, kBin = kBrz + 2 * kRH * 4, kBhn = kBin + kRH * 4, kBh = kBhn + kRH * 4;
constexpr uint32_t kRecImage = kBh + 32;
static_assert(kRecImage % 16 == 0, "bulk copy");

constexpr uint32_t kColE = 0, kColRZ = 64, kColIn = 192, kColHn = 256, kRecTmem = 512;  // the heads reuse kColE

template <int N>
struct RecTcSmem {
  static constexpr int D = kObsFixed + N;
  alignas(128) unsigned char img[(kRecImage + 127) / 128 * 128];
  alignas(128) unsigned char a[(kTileRows / 8) * (kRK1 / 8) * kALbo];  // bf16 observations (padded core-matrix pitch)
  alignas(128) unsigned char emb[kTileRows * kRH * 2];                 // bf16 embedding; the bootstrap step's h'
  alignas(128) unsigned char hid[kTileRows * kRH * 2];                 // bf16 hidden vectors, carried
  alignas(128) float stage[kTileRows * D];                             // fp32 observation block in the global layout
  alignas(8) uint64_t load_bar, mma_bar;
  uint32_t tmem_base;
};

__global__ void prep_rec_tc_kernel(const float *__restrict__ params, unsigned char *__restrict__ image, ParamLayout L, int D) {
  auto bf = [&](uint32_t off) { return reinterpret_cast<__nv_bfloat16 *>(image + off); };
  const int tid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
  for (int i = tid; i < kRH * kRK1; i += nth) {
    const int n = i / kRK1, k = i - n * kRK1;
    bf(kW1)[canon_offset(n, k, kRK1) / 2] = __float2bfloat16_rn(k < D ? params[L.W1 + static_cast<size_t>(n) * D + k] : 0.0f);
  }
  for (int i = tid; i < 3 * kRH * kRH; i += nth) {
    const int n = i / kRH, k = i - n * kRH;
    bf(kWih)[canon_offset(n, k, kRH) / 2] = __float2bfloat16_rn(params[L.Wih + i]);
    bf(kWhh)[canon_offset(n, k, kRH) / 2] = __float2bfloat16_rn(params[L.Whh + i]);
  }
  for (int i = tid; i < kHeadRows * kRH; i += nth) {
    const int n = i / kRH, k = i - n * kRH;
    float v = 0.0f;
    if (n < kActions) v = params[L.Wa + static_cast<size_t>(n) * kRH + k];
    else if (n == kActions) v = params[L.Wv + k];
    bf(kWh)[canon_offset(n, k, kRH) / 2] = __float2bfloat16_rn(v);
  }
  float *b1 = reinterpret_cast<float *>(image + kB1), *brz = reinterpret_cast<float *>(image + kBrz),
        *bin = reinterpret_cast<float *>(image + kBin), *bhn = reinterpret_cast<float *>(image + kBhn), *bh = reinterpret_cast<float *>(image + kBh);
  for (int i = tid; i < kRH; i += nth) {
    b1[i] = params[L.b1 + i];
    brz[i] = params[L.bih + i] + params[L.bhh + i];                      // r: both parts' biases
    brz[kRH + i] = params[L.bih + kRH + i] + params[L.bhh + kRH + i];    // z
    bin[i] = params[L.bih + 2 * kRH + i];
    bhn[i] = params[L.bhh + 2 * kRH + i];
  }
  if (tid < 8) bh[tid] = tid < kActions ? params[L.ba + tid] : (tid == kActions ? params[L.bv] : 0.0f);
}

__device__ __forceinline__ uint64_t rdesc(uint32_t tile, int C, int k) { return smem_desc(tile + k * 256, 128, C * 16); }
// Branch-free forms (ex2.approx and rcp.approx: a few 1e-7, far below the bf16 step the result is rounded to), so
// that the compiler can interleave the units of a row: with one warp per scheduler the gate epilogue is bound by
// the latency of dependent instructions, not by their number.
// The arguments are clamped to where the functions have long saturated in binary32, which keeps the exponential finite.
__device__ __forceinline__ float sigm(float v) { return __fdividef(1.0f, 1.0f + __expf(-fminf(fmaxf(v, -30.0f), 30.0f))); }
__device__ __forceinline__ float tanh_fast(float v) { return 1.0f - __fdividef(2.0f, 1.0f + __expf(2.0f * fminf(fmaxf(v, -15.0f), 15.0f))); }
__device__ __forceinline__ uint4 lds_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

template <int N, int F>
__global__ void __launch_bounds__(kGroupThreads, 1)
rollout_rec_tc_kernel(RolloutArgs a, const unsigned char *__restrict__ image, float *__restrict__ hidden, int ept, int n_tiles) {
  constexpr int D = kObsFixed + N, K1 = kRK1, H = kRH;
  constexpr int EPW = 32 / N, RPW = EPW * N;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  RecTcSmem<N> &sm = *reinterpret_cast<RecTcSmem<N> *>(smem_raw);
  const int row = threadIdx.x, warp = row >> 5, lane = row & 31;
  const uint32_t load_bar = smem_u32(&sm.load_bar), bar = smem_u32(&sm.mma_bar);
  if (row == 0) {
    mbar_init(load_bar, 1); mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)), "r"(kRecTmem) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  const uint32_t a_addr = smem_u32(sm.a), emb_addr = smem_u32(sm.emb), hid_addr = smem_u32(sm.hid), stage_addr = smem_u32(sm.stage);
  for (int i = row; i < static_cast<int>(sizeof(sm.a) / 16); i += kGroupThreads) sts_zero16(a_addr + 16u * i);
  for (int i = row; i < static_cast<int>((sizeof(sm.stage) + 15) / 16); i += kGroupThreads) sts_zero16(stage_addr + 16u * i);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (row == 0) {
    mbar_expect_tx(load_bar, kRecImage);
    for (uint32_t o = 0; o < kRecImage; o += 16384) bulk_load(smem_u32(sm.img + o), image + o, min(16384u, kRecImage - o), load_bar);
  }
  bool timed_out = !mbar_wait(load_bar, 0);
  timed_out = __syncthreads_or(timed_out) != 0;

  const uint32_t tmem = sm.tmem_base;
  const uint32_t lane_off = static_cast<uint32_t>(warp * 32) << 16;
  const uint32_t w1 = smem_u32(sm.img + kW1), wih = smem_u32(sm.img + kWih), whh = smem_u32(sm.img + kWhh), wh = smem_u32(sm.img + kWh);
  const float *b1 = reinterpret_cast<const float *>(sm.img + kB1), *brz = reinterpret_cast<const float *>(sm.img + kBrz),
              *bin = reinterpret_cast<const float *>(sm.img + kBin), *bhn = reinterpret_cast<const float *>(sm.img + kBhn),
              *bhd = reinterpret_cast<const float *>(sm.img + kBh);
  const uint32_t my_hid = hid_addr + static_cast<uint32_t>((row >> 3) * (H * 16) + (row & 7) * 16);  // chunk c of this row: + 128 c
  const uint32_t my_emb = emb_addr + static_cast<uint32_t>((row >> 3) * (H * 16) + (row & 7) * 16);
  uint32_t phase = 0;
  bool bulk_pending = false;
  const size_t M = static_cast<size_t>(a.env.n_envs) * N;
  const int le = warp * EPW + lane / N, ag = lane % N, crow = le * N + ag;

  for (int it = 0; !timed_out; ++it) {
    const int tile = it * static_cast<int>(gridDim.x) + static_cast<int>(blockIdx.x);
    if (tile >= n_tiles) break;
    const int e0 = tile * ept;
    const int n_env = min(ept, a.env.n_envs - e0);
    const int n_rows = n_env * N;
    const bool active = lane < RPW && le < n_env;
    const int base = active ? lane - ag : lane;
    const uint32_t env_id = static_cast<uint32_t>(a.env.first_env + e0 + le);
    EnvRegs<N, F> env;
    if (active) {
      load_env(env, a.state[e0 + le]);
    } else {
#pragma unroll
      for (int k = 0; k < N + F; ++k) env.ent[k] = 0;
      env.step = 0; env.episode = 0; env.total = 1;
    }
    {  // this row's hidden vector into the hidden tile (a carried state is a bf16 number: the conversion is exact)
      const float *src = hidden + (static_cast<size_t>(e0) * N + crow) * H;
#pragma unroll
      for (int c = 0; c < H / 8; ++c) {
        uint32_t pk[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) pk[e] = active ? pack_bf16(src[8 * c + 2 * e], src[8 * c + 2 * e + 1]) : 0u;
        sts_v4(my_hid + 128u * c, pk[0], pk[1], pk[2], pk[3]);
      }
    }
    for (int t = 0; t <= a.T; ++t) {
      const bool last = t == a.T;
      const size_t row0 = static_cast<size_t>(t) * M + static_cast<size_t>(e0) * N;
      // 1. observation
      if (active) {
        const uint32_t a_row = a_addr + a_offset<K1>(row, 0);
        observe_env<N, F>(env, a.env, ag, [&](int j, float v) {
          sts_f32(stage_addr + 4u * static_cast<uint32_t>(crow * D + j), v);
          sts_u16(a_row + a_offset<K1>(0, j), bf16_bits(v));
        });
      }
      fence_async_smem();
      tc_fence_before();
      __syncthreads();
      // 2. embedding pre-activation; hidden part of the gates
      if (row == 0) {
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < K1 / 16; ++k)
          mma_bf16(tmem + kColE, smem_desc(a_addr + k * 2 * kALbo, kALbo, (K1 / 8) * kALbo), rdesc(w1, K1, k), instr_desc(kTileRows, H), k > 0);
        mma_commit(bar);
#pragma unroll
        for (int k = 0; k < H / 16; ++k) {
          mma_bf16(tmem + kColRZ, rdesc(hid_addr, H, k), rdesc(whh, H, k), instr_desc(kTileRows, 2 * H), k > 0);
          mma_bf16(tmem + kColHn, rdesc(hid_addr, H, k), rdesc(whh + 2 * H * H * 2, H, k), instr_desc(kTileRows, H), k > 0);
        }
      }
      if (!last) {  // the observation block of this step goes out while the MMAs run
        float *obs_dst = a.buf.obs + row0 * D;
        const int count = n_rows * D;
        if (((row0 * D) & 3) == 0 && (count & 3) == 0) {
          if (row == 0) { bulk_store(obs_dst, stage_addr, static_cast<uint32_t>(count) * 4u); bulk_pending = true; }
        } else {
          for (int i = row; i < count; i += kGroupThreads) obs_dst[i] = sm.stage[i];
        }
      }
      float u = 0.0f;
      if (active && !last) u = action_uniform(a.env, a.t_global0 + static_cast<uint32_t>(t), env_id, static_cast<uint32_t>(ag));
      timed_out |= !mbar_wait(bar, phase); phase ^= 1;
      tc_fence_after();
      // 3. e = relu(. + b1) as a bf16 tile; the A tile's entries are zeroed for the next step
      {
        uint32_t ra[32], rb[32];
        tmem_ld32_nowait(tmem + kColE + lane_off, ra);
        tmem_ld32_nowait(tmem + kColE + lane_off + 32u, rb);
        tmem_ld_wait();
#pragma unroll
        for (int c = 0; c < H / 8; ++c) {
          uint32_t pk[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int j = 8 * c + 2 * e;
            const float v0 = __uint_as_float(j < 32 ? ra[j] : rb[j - 32]) + b1[j], v1 = __uint_as_float(j < 32 ? ra[j + 1] : rb[j - 31]) + b1[j + 1];
            pk[e] = relu_pack_bf16(__float_as_uint(v0), __float_as_uint(v1));
          }
          sts_v4(my_emb + 128u * c, pk[0], pk[1], pk[2], pk[3]);
        }
      }
#pragma unroll
      for (int kc = 0; kc < K1 / 8; ++kc) sts_zero16(a_addr + a_offset<K1>(row, kc * 8));
      fence_async_smem();
      tc_fence_before();
      __syncthreads();
      if (row == 0) {
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < H / 16; ++k) {
          mma_bf16(tmem + kColRZ, rdesc(emb_addr, H, k), rdesc(wih, H, k), instr_desc(kTileRows, 2 * H), 1);
          mma_bf16(tmem + kColIn, rdesc(emb_addr, H, k), rdesc(wih + 2 * H * H * 2, H, k), instr_desc(kTileRows, H), k > 0);
        }
        mma_commit(bar);
      }
      if (bulk_pending) { bulk_store_wait_read(); bulk_pending = false; }  // thread 0: the block has been read
      timed_out |= !mbar_wait(bar, phase); phase ^= 1;
      tc_fence_after();
      // 4. gates (fp32) and the new hidden vector
      {
        const uint32_t dst = last ? my_emb : my_hid;
#pragma unroll
        for (int c0 = 0; c0 < H; c0 += 16) {
          float gr[16], gz[16], gi[16], gh[16];
          tmem_ld16(tmem + kColRZ + lane_off + static_cast<uint32_t>(c0), gr);
          tmem_ld16(tmem + kColRZ + lane_off + static_cast<uint32_t>(H + c0), gz);
          tmem_ld16(tmem + kColIn + lane_off + static_cast<uint32_t>(c0), gi);
          tmem_ld16(tmem + kColHn + lane_off + static_cast<uint32_t>(c0), gh);
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            const uint4 hp = lds_v4(my_hid + 128u * static_cast<uint32_t>(c0 / 8 + c));
            const uint32_t hw[4] = {hp.x, hp.y, hp.z, hp.w};
            uint32_t pk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              float hn[2];
#pragma unroll
              for (int s = 0; s < 2; ++s) {
                const int q = 8 * c + 2 * e + s, j = c0 + q;
                const float hprev = __uint_as_float(s == 0 ? (hw[e] << 16) : (hw[e] & 0xFFFF0000u));
                const float r = sigm(gr[q] + brz[j]);
                const float z = sigm(gz[q] + brz[H + j]);
                const float n = tanh_fast(gi[q] + bin[j] + r * (gh[q] + bhn[j]));
                hn[s] = (1.0f - z) * n + z * hprev;
              }
              pk[e] = pack_bf16(hn[0], hn[1]);
            }
            sts_v4(dst + 128u * static_cast<uint32_t>(c0 / 8 + c), pk[0], pk[1], pk[2], pk[3]);
          }
        }
      }
      fence_async_smem();
      tc_fence_before();
      __syncthreads();
      // the fp32 block is zeroed for the next step: its copy has been read (thread 0 waited for that before it arrived
      // at the barrier above); the barrier after the sampler orders the zeros before the next observation
      for (int i = row; i < static_cast<int>((sizeof(sm.stage) + 15) / 16); i += kGroupThreads) sts_zero16(stage_addr + 16u * i);
      // 5. heads on the new hidden vectors
      if (row == 0) {
        tc_fence_after();
        const uint32_t src = last ? emb_addr : hid_addr;
#pragma unroll
        for (int k = 0; k < H / 16; ++k) mma_bf16(tmem + kColE, rdesc(src, H, k), rdesc(wh, H, k), instr_desc(kTileRows, kHeadRows), k > 0);
        mma_commit(bar);
      }
      timed_out |= !mbar_wait(bar, phase); phase ^= 1;
      tc_fence_after();
      int action = 0;
      float hv[16];
      tmem_ld16(tmem + kColE + lane_off, hv);
#pragma unroll
      for (int k = 0; k <= kActions; ++k) hv[k] += bhd[k];
      if (active) {
        a.buf.values[row0 + crow] = hv[kActions];
        if (!last) {
          float e[kActions];
          float m = hv[0];
#pragma unroll
          for (int k = 1; k < kActions; ++k) m = fmaxf(m, hv[k]);
          float sum = 0.0f;
#pragma unroll
          for (int k = 0; k < kActions; ++k) { e[k] = __expf(hv[k] - m); sum += e[k]; }
          const float target = u * sum;
          action = kActions - 1;
          float cdf = 0.0f;
          bool found = false;
#pragma unroll
          for (int k = 0; k < kActions; ++k) {
            cdf += e[k];
            if (!found && target < cdf) { action = k; found = true; }
          }
          if (a.forced) {
            action = a.forced[row0 + crow];
            if (action < 0 || action >= kActions) action = 0;
          }
          float la = hv[0];
#pragma unroll
          for (int k = 1; k < kActions; ++k) la = (action == k) ? hv[k] : la;
          a.buf.actions[row0 + crow] = action;
          a.buf.logp[row0 + crow] = la - m - __logf(sum);
          if (a.write_logits) {
#pragma unroll
            for (int k = 0; k < kActions; ++k) a.buf.logits[(row0 + crow) * kActions + k] = hv[k];
          }
        }
      }
      tc_fence_before();
      if (__syncthreads_or(timed_out)) { timed_out = true; break; }
      if (last) break;
      float reward;
      bool done;
      step_env_warp<N, F>(env, a.env, env_id, ag, base, active, action, reward, done);
      if (active) {
        a.buf.rewards[row0 + crow] = reward;
        if (ag == 0) a.buf.dones[static_cast<size_t>(t) * a.env.n_envs + e0 + le] = done ? 1 : 0;
        if (done) {  // a finished episode leaves no memory behind
#pragma unroll
          for (int c = 0; c < H / 8; ++c) sts_zero16(my_hid + 128u * c);
        }
      }
    }
    if (!timed_out && active) {
      float *dst = hidden + (static_cast<size_t>(e0) * N + crow) * H;
#pragma unroll
      for (int c = 0; c < H / 8; ++c) {
        const uint4 hp = lds_v4(my_hid + 128u * c);
        const uint32_t hw[4] = {hp.x, hp.y, hp.z, hp.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          dst[8 * c + 2 * e] = __uint_as_float(hw[e] << 16);
          dst[8 * c + 2 * e + 1] = __uint_as_float(hw[e] & 0xFFFF0000u);
        }
      }
      if (ag == 0) store_env(env, a.state[e0 + le]);
    }
    __syncthreads();  // the hidden tile is rewritten by the next tile's rows
  }
  if (timed_out && row == 0) atomicExch(a.status, kStatusTimeout);
  bulk_store_wait_all();
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kRecTmem) : "memory");
  }
}

template <int N, int F>
cudaError_t launch_rec_tc_variant(mava_rollout *h, const RolloutArgs &args) {
  constexpr int D = kObsFixed + N, EPT_MAX = 4 * (32 / N);
  auto kern = rollout_rec_tc_kernel<N, F>;
  const size_t smem = sizeof(RecTcSmem<N>);
  cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (err != cudaSuccess) return err;
  int sms = 0;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->device);
  if (err != cudaSuccess) return err;
  int ept = (h->cfg.n_envs + sms - 1) / sms;
  if (ept > EPT_MAX) ept = EPT_MAX;
  if (ept < 1) ept = 1;
  for (int e = ept; e <= EPT_MAX; ++e)  // a block that is a whole number of 16-byte pieces leaves as one bulk copy
    if ((e * N * D) % 4 == 0) { ept = e; break; }
  const int n_tiles = (h->cfg.n_envs + ept - 1) / ept;
  kern<<<n_tiles < sms ? n_tiles : sms, kGroupThreads, smem, h->stream>>>(args, static_cast<const unsigned char *>(h->d_wtc), h->d_hidden, ept, n_tiles);
  h->launches += 1;
  return cudaGetLastError();
}

}  // namespace

size_t rec_tc_weight_bytes(const mava_config_t &) { return kRecImage; }

cudaError_t launch_rollout_rec_tc(mava_rollout *h, const float *params_dev, const RolloutArgs &args) {
  if (h->cfg.hidden != kRH || h->D > kRK1) return cudaErrorNotSupported;
  prep_rec_tc_kernel<<<32, 256, 0, h->stream>>>(params_dev, static_cast<unsigned char *>(h->d_wtc), param_layout(h->cfg, h->D, 1), h->D);
  h->launches += 1;
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  switch (h->variant) {
    case 5: return launch_rec_tc_variant<2, 2>(h, args);
    case 6: return launch_rec_tc_variant<3, 3>(h, args);
    default: return cudaErrorNotSupported;
  }
}

}  // namespace mava
