// bf16 tensor-core rollout for sm_100a: tcgen05.mma with fp32 accumulators in tensor memory.
//
// One persistent CTA per SM keeps the bf16 weights resident in shared memory (loaded once with
// bulk async copies, in the canonical K-major core-matrix layout the MMA reads) and runs
// kGroups independent groups of 128 threads.  A group owns one tile of environments (up to 128
// agent rows = the M of the MMA) for all T steps, then takes its next tile.  Per step a group
//   1. writes the non-zero entries of its observation rows over a zero background (fp32),
//   2. copies that block to the time-major obs array and re-packs it as the bf16 A operand,
//   3. runs layer 1, layer 2 and the heads as three MMAs (thread 0 issues; completion arrives on
//      an mbarrier), each followed by an epilogue out of tensor memory: thread r owns row r
//      (bias, ReLU, bf16, store as the next A operand; for the heads: softmax, Philox draw,
//      inverse-CDF action, log-prob),
//   4. applies the transition and auto-reset.
// Groups never wait for one another, so while one group sits in an MMA or a tensor-memory
// round trip the other fills the SM.  Every wait on an mbarrier is bounded: when it runs out
// the group records kStatusTimeout, stops stepping and falls through to the common exit.
#include <cuda_bf16.h>

#include "common.cuh"
#include "env.cuh"
#include "layout.h"

namespace mava {
namespace {

constexpr int kGroups = 2;
constexpr int kGroupThreads = 128;
constexpr int kTcThreads = kGroups * kGroupThreads;
constexpr int kTileRows = 128;       // M of every MMA
constexpr int kHeadRows = 16;        // heads padded to the smallest N the MMA takes at M = 128
constexpr uint32_t kSpinLimit = 1u << 22;

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait; false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kSpinLimit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void group_sync(int g) {
  asm volatile("bar.sync %0, %1;" ::"r"(g + 1), "r"(kGroupThreads) : "memory");
}
// Barrier of the group that also ORs a predicate over its threads.
__device__ __forceinline__ bool group_any(int g, bool pred) {
  uint32_t out;
  asm volatile(
      "{\n.reg .pred p, q;\n"
      "setp.ne.u32 p, %1, 0;\n"
      "barrier.cta.red.or.pred q, %2, %3, p;\n"
      "selp.u32 %0, 1, 0, q;\n}"
      : "=r"(out)
      : "r"(static_cast<uint32_t>(pred)), "r"(g + 1), "r"(kGroupThreads)
      : "memory");
  return out != 0;
}

// Shared-memory matrix descriptor, no swizzle, K-major: core matrices of 8 rows x 16 bytes;
// lbo = byte step between core matrices along K, sbo = byte step between 8-row groups.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>((lbo >> 4) & 0x3FFFu) << 16) |
         (static_cast<uint64_t>((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}
// Instruction descriptor of kind::f16: fp32 accumulate, bf16 A and B, both K-major, M x N.
__host__ __device__ constexpr uint32_t instr_desc(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(m >> 4) << 24);
}
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 32 bit, 16 consecutive columns: thread i of the warp reads lane (lane base + i).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float *v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);  // .x = lo (low half), .y = hi
  return *reinterpret_cast<const uint32_t *>(&b);
}

// ---- shapes ------------------------------------------------------------------------------------
template <int N, int H>
struct TcShape {
  static constexpr int D = kObsFixed + N;
  static constexpr int K1 = (D + 15) / 16 * 16;               // layer-1 K padded to the MMA's K step
  static constexpr int EPT_MAX = kTileRows / N;                // environments per tile, at most
  static constexpr uint32_t W1_BYTES = H * K1 * 2, W2_BYTES = H * H * 2, WH_BYTES = kHeadRows * H * 2;
  static constexpr uint32_t BIAS_FLOATS = 2 * H + kHeadRows;
  static constexpr uint32_t IMAGE_BYTES = W1_BYTES + W2_BYTES + WH_BYTES + BIAS_FLOATS * 4;
  static constexpr uint32_t STAGE_BYTES = (kTileRows * D * 4 + 15) / 16 * 16;
  static constexpr uint32_t AH_BYTES = kTileRows * (K1 > H ? K1 : H) * 2;
  static constexpr int ACC_COLS = H;                            // layer accumulators (reused)
  static constexpr int GROUP_COLS = H + 32;                     // + the heads accumulator
  static constexpr int TMEM_COLS = kGroups * GROUP_COLS <= 256 ? 256 : 512;
};

template <int N, int F, int H>
struct TcGroupSmem {
  using S = TcShape<N, H>;
  alignas(16) unsigned char stage[S::STAGE_BYTES];  // fp32 observation block, global layout
  alignas(128) unsigned char ah[S::AH_BYTES];       // A operand: observations, then h1, then h2
  EnvRec st[S::EPT_MAX];
  int act[kTileRows];
  uint8_t new_r[kTileRows], new_c[kTileRows], collected[S::EPT_MAX * F];
  alignas(8) uint64_t mma_bar;
};

template <int N, int F, int H>
struct TcSmem {
  using S = TcShape<N, H>;
  alignas(128) unsigned char weights[S::IMAGE_BYTES];  // W1 | W2 | heads | b1 b2 bh (fp32)
  TcGroupSmem<N, F, H> grp[kGroups];
  alignas(8) uint64_t load_bar;
  uint32_t tmem_base;
};

// ---- weight image ------------------------------------------------------------------------------
// Byte offset of element (n, k) of an N x K bf16 operand in the canonical no-swizzle K-major
// layout used here: 8-row groups are K*16 bytes apart, core matrices along K 128 bytes apart.
__host__ __device__ constexpr uint32_t canon_offset(int n, int k, int K) {
  return static_cast<uint32_t>((n >> 3) * (K * 16) + (k >> 3) * 128 + (n & 7) * 16 + (k & 7) * 2);
}

template <int N, int H>
__global__ void prep_tc_kernel(const float *__restrict__ params, unsigned char *__restrict__ image, ParamLayout L) {
  using S = TcShape<N, H>;
  constexpr int D = S::D, K1 = S::K1;
  __nv_bfloat16 *w1 = reinterpret_cast<__nv_bfloat16 *>(image);
  __nv_bfloat16 *w2 = reinterpret_cast<__nv_bfloat16 *>(image + S::W1_BYTES);
  __nv_bfloat16 *wh = reinterpret_cast<__nv_bfloat16 *>(image + S::W1_BYTES + S::W2_BYTES);
  float *bias = reinterpret_cast<float *>(image + S::W1_BYTES + S::W2_BYTES + S::WH_BYTES);
  const int tid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
  for (int i = tid; i < H * K1; i += nth) {
    const int n = i / K1, k = i - n * K1;
    w1[canon_offset(n, k, K1) / 2] = __float2bfloat16_rn(k < D ? params[L.W1 + static_cast<size_t>(n) * D + k] : 0.0f);
  }
  for (int i = tid; i < H * H; i += nth) {
    const int n = i / H, k = i - n * H;
    w2[canon_offset(n, k, H) / 2] = __float2bfloat16_rn(params[L.W2 + static_cast<size_t>(n) * H + k]);
  }
  for (int i = tid; i < kHeadRows * H; i += nth) {
    const int n = i / H, k = i - n * H;
    float v = 0.0f;
    if (n < kActions) v = params[L.Wa + static_cast<size_t>(n) * H + k];
    else if (n == kActions) v = params[L.Wv + k];
    wh[canon_offset(n, k, H) / 2] = __float2bfloat16_rn(v);
  }
  for (int i = tid; i < static_cast<int>(S::BIAS_FLOATS); i += nth) {
    float v = 0.0f;
    if (i < H) v = params[L.b1 + i];
    else if (i < 2 * H) v = params[L.b2 + i - H];
    else if (i - 2 * H < kActions) v = params[L.ba + i - 2 * H];
    else if (i - 2 * H == kActions) v = params[L.bv];
    bias[i] = v;
  }
}

// ---- the rollout kernel ------------------------------------------------------------------------
// Epilogue of a hidden layer: thread `row` reads its accumulator row from tensor memory, adds the
// bias, applies ReLU, rounds to bf16 and stores the row as the next A operand (K = H).
template <int H>
__device__ __forceinline__ void hidden_epilogue(uint32_t acc_taddr, const float *bias, unsigned char *ah, int row) {
#pragma unroll 1
  for (int c0 = 0; c0 < H; c0 += 16) {
    float v[16];
    tmem_ld16(acc_taddr + static_cast<uint32_t>(c0), v);
    uint32_t packed[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float a = fmaxf(v[2 * i] + bias[c0 + 2 * i], 0.0f);
      const float b = fmaxf(v[2 * i + 1] + bias[c0 + 2 * i + 1], 0.0f);
      packed[i] = pack_bf16(a, b);
    }
    uint4 *dst0 = reinterpret_cast<uint4 *>(ah + canon_offset(row, c0, H));
    uint4 *dst1 = reinterpret_cast<uint4 *>(ah + canon_offset(row, c0 + 8, H));
    *dst0 = make_uint4(packed[0], packed[1], packed[2], packed[3]);
    *dst1 = make_uint4(packed[4], packed[5], packed[6], packed[7]);
  }
}

template <int N, int F, int H>
__global__ void __launch_bounds__(kTcThreads, 1)
rollout_tc_kernel(RolloutArgs a, const unsigned char *__restrict__ image, int ept, int n_tiles) {
  using S = TcShape<N, H>;
  constexpr int D = S::D, K1 = S::K1;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  TcSmem<N, F, H> &sm = *reinterpret_cast<TcSmem<N, F, H> *>(smem_raw);
  const int tid = threadIdx.x;
  const int g = tid / kGroupThreads;   // group index
  const int row = tid % kGroupThreads; // row of the tile this thread owns; also its TMEM lane
  const int warp = tid / 32;
  TcGroupSmem<N, F, H> &gs = sm.grp[g];

  // ---- one-time set-up: barriers, tensor memory, weights -------------------------------------
  if (tid == 0) {
    mbar_init(smem_u32(&sm.load_bar), 1);
    for (int i = 0; i < kGroups; ++i) mbar_init(smem_u32(&sm.grp[i].mma_bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                 "r"(S::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  {  // zero the observation block and the A operand once (the block keeps a zero background)
    uint4 *z = reinterpret_cast<uint4 *>(gs.stage);
    for (int i = row; i < static_cast<int>(S::STAGE_BYTES / 16); i += kGroupThreads) z[i] = make_uint4(0, 0, 0, 0);
    z = reinterpret_cast<uint4 *>(gs.ah);
    for (int i = row; i < static_cast<int>(S::AH_BYTES / 16); i += kGroupThreads) z[i] = make_uint4(0, 0, 0, 0);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  bool timed_out = false;
  if (tid == 0) {
    const uint32_t bar = smem_u32(&sm.load_bar);
    mbar_expect_tx(bar, S::IMAGE_BYTES);
    constexpr uint32_t kChunk = 16384;
    for (uint32_t off = 0; off < S::IMAGE_BYTES; off += kChunk) {
      const uint32_t n = S::IMAGE_BYTES - off < kChunk ? S::IMAGE_BYTES - off : kChunk;
      bulk_load(smem_u32(sm.weights + off), image + off, n, bar);
    }
  }
  timed_out = !mbar_wait(smem_u32(&sm.load_bar), 0);
  timed_out = __syncthreads_or(timed_out) != 0;  // uniform: the tile loops below depend on it

  const uint32_t tmem_base = sm.tmem_base;
  const uint32_t acc_col = tmem_base + static_cast<uint32_t>(g * S::GROUP_COLS);
  const uint32_t head_col = acc_col + static_cast<uint32_t>(S::ACC_COLS);
  const uint32_t lane_off = static_cast<uint32_t>((warp % 4) * 32) << 16;  // this warp's TMEM lanes
  const uint32_t w1_addr = smem_u32(sm.weights), w2_addr = w1_addr + S::W1_BYTES, wh_addr = w2_addr + S::W2_BYTES;
  const float *bias = reinterpret_cast<const float *>(sm.weights + S::W1_BYTES + S::W2_BYTES + S::WH_BYTES);
  const uint32_t ah_addr = smem_u32(gs.ah);
  const uint32_t bar = smem_u32(&gs.mma_bar);
  float *stage = reinterpret_cast<float *>(gs.stage);
  uint32_t phase = 0;
  const size_t M = static_cast<size_t>(a.env.n_envs) * N;

  // ---- tiles of this group ---------------------------------------------------------------------
  for (int tile = blockIdx.x * kGroups + g; tile < n_tiles && !timed_out; tile += gridDim.x * kGroups) {
    const int e0 = tile * ept;
    const int n_env = min(ept, a.env.n_envs - e0);
    const int n_rows = n_env * N;
    for (int i = row; i < n_env * static_cast<int>(sizeof(EnvRec) / 4); i += kGroupThreads)
      reinterpret_cast<uint32_t *>(gs.st)[i] = reinterpret_cast<const uint32_t *>(a.state + e0)[i];
    group_sync(g);
    const int le = row / N, ag = row - le * N;  // this thread's environment and agent (if row < n_rows)

    for (int t = 0; t <= a.T; ++t) {
      const bool last = (t == a.T);
      const size_t row0 = static_cast<size_t>(t) * M + static_cast<size_t>(e0) * N;
      // 1. non-zero observation entries over the zero background
      if (row < n_rows)
        observe_sparse<N, F>(gs.st[le], a.env, ag, [&](int j, float v) { stage[row * D + j] = v; });
      group_sync(g);
      // 2a. observation block -> obs[t] (one contiguous block of the time-major array)
      if (!last) {
        float *dst = a.buf.obs + row0 * D;
        const int count = n_rows * D;
        if (((row0 * D) & 3) == 0 && (count & 3) == 0) {
          for (int i = row; i < count / 4; i += kGroupThreads)
            reinterpret_cast<float4 *>(dst)[i] = reinterpret_cast<const float4 *>(stage)[i];
        } else {
          for (int i = row; i < count; i += kGroupThreads) dst[i] = stage[i];
        }
      }
      // 2b. the same rows as the bf16 A operand of layer 1 (K padded with zeros)
      if (row < n_rows) {
#pragma unroll
        for (int kc = 0; kc < K1 / 8; ++kc) {
          float x[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) x[i] = (kc * 8 + i < D) ? stage[row * D + kc * 8 + i] : 0.0f;
          *reinterpret_cast<uint4 *>(gs.ah + canon_offset(row, kc * 8, K1)) =
              make_uint4(pack_bf16(x[0], x[1]), pack_bf16(x[2], x[3]), pack_bf16(x[4], x[5]), pack_bf16(x[6], x[7]));
        }
      }
      fence_async_smem();
      tc_fence_before();
      group_sync(g);
      // 3. layer 1; meanwhile the other threads restore the zero background
      if (row == 0) {
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < K1 / 16; ++k)
          mma_bf16(acc_col, smem_desc(ah_addr + k * 256, 128, K1 * 16), smem_desc(w1_addr + k * 256, 128, K1 * 16),
                   instr_desc(kTileRows, H), k > 0);
        mma_commit(bar);
      }
      if (row < n_rows) observe_sparse<N, F>(gs.st[le], a.env, ag, [&](int j, float) { stage[row * D + j] = 0.0f; });
      timed_out |= !mbar_wait(bar, phase);
      phase ^= 1;
      tc_fence_after();
      hidden_epilogue<H>(acc_col + lane_off, bias, gs.ah, row);
      fence_async_smem();
      tc_fence_before();
      group_sync(g);
      // 4. layer 2
      if (row == 0) {
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < H / 16; ++k)
          mma_bf16(acc_col, smem_desc(ah_addr + k * 256, 128, H * 16), smem_desc(w2_addr + k * 256, 128, H * 16),
                   instr_desc(kTileRows, H), k > 0);
        mma_commit(bar);
      }
      timed_out |= !mbar_wait(bar, phase);
      phase ^= 1;
      tc_fence_after();
      hidden_epilogue<H>(acc_col + lane_off, bias + H, gs.ah, row);
      fence_async_smem();
      tc_fence_before();
      group_sync(g);
      // 5. heads: six logits and the value, N padded to 16
      if (row == 0) {
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < H / 16; ++k)
          mma_bf16(head_col, smem_desc(ah_addr + k * 256, 128, H * 16), smem_desc(wh_addr + k * 256, 128, H * 16),
                   instr_desc(kTileRows, kHeadRows), k > 0);
        mma_commit(bar);
      }
      timed_out |= !mbar_wait(bar, phase);
      phase ^= 1;
      tc_fence_after();
      {
        float hv[16];
        tmem_ld16(head_col + lane_off, hv);
        if (row < n_rows) {
          const float *bh = bias + 2 * H;
          a.buf.values[row0 + row] = hv[kActions] + bh[kActions];
          if (!last) {
            float l[kActions], e[kActions];
#pragma unroll
            for (int k = 0; k < kActions; ++k) l[k] = hv[k] + bh[k];
            float m = l[0];
#pragma unroll
            for (int k = 1; k < kActions; ++k) m = fmaxf(m, l[k]);
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
              action = a.forced[row0 + row];
              if (action < 0 || action >= kActions) action = 0;
            }
            float la = l[0];
#pragma unroll
            for (int k = 1; k < kActions; ++k) la = (action == k) ? l[k] : la;
            gs.act[row] = action;
            a.buf.actions[row0 + row] = action;
            a.buf.logp[row0 + row] = la - m - logf(sum);
            if (a.write_logits) {
#pragma unroll
              for (int k = 0; k < kActions; ++k) a.buf.logits[(row0 + row) * kActions + k] = l[k];
            }
          }
        }
      }
      tc_fence_before();
      if (group_any(g, timed_out)) { timed_out = true; break; }
      if (last) break;
      // 6. transition and auto-reset
      step_decide<N, F>(gs.st, a.env, gs.act, n_env, gs.new_r, gs.new_c, gs.collected, row, kGroupThreads);
      group_sync(g);
      if (row < n_env) {
        float reward;
        bool done;
        step_apply<N, F>(gs.st[row], a.env, static_cast<uint32_t>(a.env.first_env + e0 + row), gs.new_r, gs.new_c,
                         gs.collected, row, reward, done);
        for (int n = 0; n < N; ++n) a.buf.rewards[row0 + row * N + n] = reward;
        a.buf.dones[static_cast<size_t>(t) * a.env.n_envs + e0 + row] = done ? 1 : 0;
      }
      group_sync(g);
    }
    if (!timed_out)
      for (int i = row; i < n_env * static_cast<int>(sizeof(EnvRec) / 4); i += kGroupThreads)
        reinterpret_cast<uint32_t *>(a.state + e0)[i] = reinterpret_cast<const uint32_t *>(gs.st)[i];
    group_sync(g);
  }
  if (timed_out && row == 0) atomicExch(a.status, kStatusTimeout);

  // ---- common exit: every thread arrives here; tensor memory is returned ----------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(S::TMEM_COLS) : "memory");
  }
}

template <int N, int F, int H>
cudaError_t launch_tc_variant(mava_rollout *h, const RolloutArgs &args) {
  using S = TcShape<N, H>;
  auto kern = rollout_tc_kernel<N, F, H>;
  const size_t smem = sizeof(TcSmem<N, F, H>);
  cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (err != cudaSuccess) return err;
  int sms = 0;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->device);
  if (err != cudaSuccess) return err;
  // Environments per tile: full tiles when there is enough work for every group of every SM,
  // otherwise smaller tiles so that all groups have one (the per-step chain is latency-bound).
  const int slots = sms * kGroups;
  int ept = (h->cfg.n_envs + slots - 1) / slots;
  if (ept > S::EPT_MAX) ept = S::EPT_MAX;
  if (ept < 1) ept = 1;
  const int n_tiles = (h->cfg.n_envs + ept - 1) / ept;
  const int grid = (n_tiles + kGroups - 1) / kGroups < sms ? (n_tiles + kGroups - 1) / kGroups : sms;
  kern<<<grid, kTcThreads, smem, h->stream>>>(args, static_cast<const unsigned char *>(h->d_wtc), ept, n_tiles);
  h->launches += 1;
  return cudaGetLastError();
}

template <int N, int H>
cudaError_t launch_prep_variant(mava_rollout *h, const float *params_dev) {
  prep_tc_kernel<N, H><<<64, 256, 0, h->stream>>>(params_dev, static_cast<unsigned char *>(h->d_wtc),
                                                 param_layout(h->cfg, h->D, 1));
  h->launches += 1;
  return cudaGetLastError();
}

}  // namespace

bool tc_supported(const mava_config_t &cfg) {
  const int v = find_variant(cfg);
  return v == 0 || v == 1 || v == 2;  // shared torso, H <= 128
}

size_t tc_weight_bytes(const mava_config_t &cfg, int) {
  switch (find_variant(cfg)) {
    case 0: return TcShape<2, 64>::IMAGE_BYTES;
    case 1: return TcShape<2, 128>::IMAGE_BYTES;
    case 2: return TcShape<3, 128>::IMAGE_BYTES;
    default: return 16;
  }
}

cudaError_t launch_prep_tc(mava_rollout *h, const float *params_dev) {
  switch (h->variant) {
    case 0: return launch_prep_variant<2, 64>(h, params_dev);
    case 1: return launch_prep_variant<2, 128>(h, params_dev);
    case 2: return launch_prep_variant<3, 128>(h, params_dev);
    default: return cudaErrorNotSupported;
  }
}

cudaError_t launch_rollout_tc(mava_rollout *h, const RolloutArgs &args) {
  switch (h->variant) {
    case 0: return launch_tc_variant<2, 2, 64>(h, args);
    case 1: return launch_tc_variant<2, 2, 128>(h, args);
    case 2: return launch_tc_variant<3, 3, 128>(h, args);
    default: return cudaErrorNotSupported;
  }
}

}  // namespace mava
