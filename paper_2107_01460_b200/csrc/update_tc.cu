// Update block on the tensor cores (sm_100a, tcgen05): the multi-agent PPO loss of one minibatch and its gradient for the
// shared-torso nets with H <= 128 and D <= 80, bf16 operands with fp32 accumulation in tensor memory.
//
// One persistent CTA per SM walks over tiles of 128 rows.  Every matrix of a tile lives once in shared memory as a bf16
// tile in the canonical core-matrix layout [row][feature] (core matrix = 8 rows x 16 bytes; feature chunks 128 bytes
// apart, 8-row groups C*16 bytes apart for a tile of C features).  Read with the feature index as K it is the K-major
// A operand of the per-row products (forward layers, d h = d z . W); read with the row index as K it is an MN-major
// operand of the products that sum over rows (d W = d z^T . input), so no transposed copy is ever written.  The same
// holds for the weights: W2 [out][in] is the K-major B operand of the forward layer and, read the other way, the
// MN-major B operand of d h1 = d z2 . W2.
//   per tile:  x -> z1 -> h1 -> z2 -> h2 -> logits, value -> loss and its per-row derivatives (fp32, thread = row)
//              -> d h2 -> d z2 -> d h1 -> d z1, and on the side d Wh^T += h2^T . dhead, d W2 += d z2^T . h1,
//              d W1 += d z1^T . x, d b2 += d z2^T . 1, d b1 += d z1^T . 1 (the ones are column 7 of the dhead tile).
// The weight-gradient accumulators stay in tensor memory for all tiles of the CTA and are written once, into the CTA's
// own slice of the partial-gradient array; a last kernel adds the slices in slice order (update.cu), so the gradient
// is the same bytes on every call.  Rounding points are those of the bf16-operand mode of the float64 oracle.
// A hidden width below 128 is padded with zero units (their activations, gates and gradients are exactly zero).
// MMAs are issued by one thread; tcgen05.commit tracks all MMAs issued before it, so a tile buffer may be rewritten as
// soon as a later commit has been waited for.  Every mbarrier wait is bounded.
#include <cuda_bf16.h>

#include "common.cuh"
#include "layout.h"
#include "tc_common.cuh"
#include "update_common.cuh"

namespace mava {
namespace {

constexpr int kUR = 128;        // rows per tile (M of the per-row products, K of the weight-gradient products)
constexpr int kUH = 128;        // hidden width, padded
constexpr int kUK1 = 80;        // input width, padded to the MMA's K step
constexpr int kUHeads = 16;     // six logits, the value, a column of ones, eight columns of zeros
constexpr int kUThreads = 256;  // thread = (row, column half)

// weight image: bf16 tiles W1 [H][K1], W2 [H][H], Wh [16][H]; then fp32 b1 [H], b2 [H], bh [8]
constexpr uint32_t kImgW1 = 0, kImgW2 = kImgW1 + kUH * kUK1 * 2, kImgWh = kImgW2 + kUH * kUH * 2;
constexpr uint32_t kImgB1 = kImgWh + kUHeads * kUH * 2, kImgB2 = kImgB1 + kUH * 4, kImgBh = kImgB2 + kUH * 4;
constexpr uint32_t kImgBytes = kImgBh + 32;
static_assert(kImgBytes % 16 == 0, "one bulk copy");

// tensor-memory columns
constexpr uint32_t kColAcc = 0, kColDW2 = 128, kColDW1 = 256, kColHead = 352, kColDWh = 384, kColDB2 = 416, kColDB1 = 448;
constexpr uint32_t kTmemCols = 512;

struct UtcSmem {
  alignas(128) unsigned char img[(kImgBytes + 127) / 128 * 128];
  alignas(128) unsigned char x[(kUR / 8) * (kUK1 / 8) * kALbo];  // feature chunks 144 bytes apart (see a_offset): the
                                                                 // converter's 2-byte stores then spread over the banks
  alignas(128) unsigned char h1[kUR * kUH * 2];
  alignas(128) unsigned char h2[kUR * kUH * 2];   // d z1 once h2's last reader is done
  alignas(128) unsigned char dz2[kUR * kUH * 2];
  alignas(128) unsigned char dhead[kUR * kUHeads * 2];
  alignas(128) float stage[kUR * kUK1];           // the tile's fp32 rows as they lie in the obs array (row stride D)
  long long rmap[kUR];
  float red[4][8];
  alignas(8) uint64_t bar_load, bar_mma, bar_end, bar_stage;
  uint32_t tmem_base;
};

__global__ void prep_upd_tc_kernel(const float *__restrict__ params, unsigned char *__restrict__ image, ParamLayout L, int D, int H) {
  auto bf = [&](uint32_t off) { return reinterpret_cast<__nv_bfloat16 *>(image + off); };
  const int tid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
  for (int i = tid; i < kUH * kUK1; i += nth) {
    const int n = i / kUK1, k = i - n * kUK1;
    bf(kImgW1)[canon_offset(n, k, kUK1) / 2] = __float2bfloat16_rn((n < H && k < D) ? params[L.W1 + static_cast<size_t>(n) * D + k] : 0.0f);
  }
  for (int i = tid; i < kUH * kUH; i += nth) {
    const int n = i / kUH, k = i - n * kUH;
    bf(kImgW2)[canon_offset(n, k, kUH) / 2] = __float2bfloat16_rn((n < H && k < H) ? params[L.W2 + static_cast<size_t>(n) * H + k] : 0.0f);
  }
  for (int i = tid; i < kUHeads * kUH; i += nth) {
    const int n = i / kUH, k = i - n * kUH;
    float v = 0.0f;
    if (k < H && n < kActions) v = params[L.Wa + static_cast<size_t>(n) * H + k];
    else if (k < H && n == kActions) v = params[L.Wv + k];
    bf(kImgWh)[canon_offset(n, k, kUH) / 2] = __float2bfloat16_rn(v);
  }
  float *b1 = reinterpret_cast<float *>(image + kImgB1), *b2 = reinterpret_cast<float *>(image + kImgB2),
        *bh = reinterpret_cast<float *>(image + kImgBh);
  for (int i = tid; i < kUH; i += nth) {
    b1[i] = i < H ? params[L.b1 + i] : 0.0f;
    b2[i] = i < H ? params[L.b2 + i] : 0.0f;
  }
  if (tid < 8) bh[tid] = tid < kActions ? params[L.ba + tid] : (tid == kActions ? params[L.bv] : 0.0f);
}

// Descriptor of a canonical tile of C features read with the feature index as K (step k = features 16 k ..).
__device__ __forceinline__ uint64_t desc_k(uint32_t tile, int C, int k) { return smem_desc(tile + k * 256, 128, C * 16); }
// The same tile read with the row index as K (step k = rows 16 k ..): the 8-row groups are the K groups, the feature
// chunks the MN groups: the descriptor's leading-dimension offset is then the step between K groups (C*16 bytes) and
// its stride offset the step between MN groups (128 bytes).
__device__ __forceinline__ uint64_t desc_mn(uint32_t tile, int C, int k) { return smem_desc(tile + k * 2 * C * 16, C * 16, 128); }
constexpr uint32_t kAmn = 1u << 15, kBmn = 1u << 16;  // operand is MN-major

struct Offsets { size_t W1, b1, W2, b2, Wa, ba, Wv, bv; };

__global__ void __launch_bounds__(kUThreads, 1)
ppo_net_tc_kernel(const unsigned char *__restrict__ image, UpdRows rows, UpdHyper hp, const double *__restrict__ adv_stats,
                  float *__restrict__ partial, size_t n_params, double *__restrict__ term_partial, int *status, Offsets off, int D,
                  int H) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  UtcSmem &sm = *reinterpret_cast<UtcSmem *>(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int row = tid & (kUR - 1), half = tid >> 7;
  const uint32_t bar_load = smem_u32(&sm.bar_load), bar_mma = smem_u32(&sm.bar_mma), bar_end = smem_u32(&sm.bar_end),
                 bar_stage = smem_u32(&sm.bar_stage);
  if (tid == 0) {
    mbar_init(bar_load, 1); mbar_init(bar_mma, 1); mbar_init(bar_end, 1); mbar_init(bar_stage, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // the x tile's pad columns and the dhead tile's upper eight columns stay zero for the whole run
  for (int i = tid; i < static_cast<int>(sizeof(sm.x) / 16); i += kUThreads) sts_zero16(smem_u32(sm.x) + 16u * i);
  for (int i = tid; i < static_cast<int>(sizeof(sm.dhead) / 16); i += kUThreads) sts_zero16(smem_u32(sm.dhead) + 16u * i);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (tid == 0) {
    mbar_expect_tx(bar_load, kImgBytes);
    constexpr uint32_t kChunk = 16384;
    for (uint32_t o = 0; o < kImgBytes; o += kChunk) bulk_load(smem_u32(sm.img + o), image + o, min(kChunk, kImgBytes - o), bar_load);
  }
  bool timed_out = !mbar_wait(bar_load, 0);
  timed_out = __syncthreads_or(timed_out) != 0;

  const uint32_t tmem = sm.tmem_base;
  const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
  const uint32_t w1 = smem_u32(sm.img + kImgW1), w2 = smem_u32(sm.img + kImgW2), wh = smem_u32(sm.img + kImgWh);
  const uint32_t xt = smem_u32(sm.x), h1t = smem_u32(sm.h1), h2t = smem_u32(sm.h2), dz2t = smem_u32(sm.dz2), dz1t = h2t,
                 dht = smem_u32(sm.dhead);
  const float *b1 = reinterpret_cast<const float *>(sm.img + kImgB1), *b2 = reinterpret_cast<const float *>(sm.img + kImgB2),
              *bh = reinterpret_cast<const float *>(sm.img + kImgBh);
  const float mean = static_cast<float>(adv_stats[0]);
  const float inv_std = 1.0f / (static_cast<float>(adv_stats[1]) + 1e-8f);
  const float inv_n = 1.0f / static_cast<float>(rows.n);
  const long long n_tiles = (rows.n + kUR - 1) / kUR;
  const int my_tiles = blockIdx.x < n_tiles ? static_cast<int>((n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0;
  auto tile_of = [&](int i) { return static_cast<long long>(blockIdx.x) + static_cast<long long>(i) * gridDim.x; };
  // a full tile of consecutive rows is one 16-byte aligned block of the obs array: it comes in by one bulk copy
  auto bulk_ok = [&](int i) { return i < my_tiles && rows.env_ids == nullptr && (tile_of(i) + 1) * kUR <= rows.n; };
  const uint32_t stage_bytes = static_cast<uint32_t>(kUR * D * 4);
  auto request_stage = [&](int i) {
    mbar_expect_tx(bar_stage, stage_bytes);
    const float *src = rows.x + static_cast<size_t>(tile_of(i)) * kUR * D;
    for (uint32_t o = 0; o < stage_bytes; o += 16384)
      bulk_load(smem_u32(sm.stage) + o, reinterpret_cast<const unsigned char *>(src) + o, min(16384u, stage_bytes - o), bar_stage);
  };
  bool stage_pending = false;  // thread 0
  if (tid == 0 && !timed_out && bulk_ok(0)) { request_stage(0); stage_pending = true; }

  uint32_t ph_mma = 0, ph_end = 0, ph_stage = 0;
  double t_actor = 0.0, t_ent = 0.0, t_value = 0.0;
  float gbh = 0.0f;  // threads 0..6: gradient of the heads' biases

  // hidden-layer epilogue: this thread's 64 accumulator columns + bias -> ReLU -> bf16 -> its row of `dst`; returns
  // the gate bits (bit c: unit 64 half + c is active)
  auto fwd_epilogue = [&](const float *bias, uint32_t dst) -> uint64_t {
    uint32_t ra[32], rb[32];
    tmem_ld32_nowait(tmem + kColAcc + lane_off + 64u * half, ra);
    tmem_ld32_nowait(tmem + kColAcc + lane_off + 64u * half + 32u, rb);
    tmem_ld_wait();
    uint64_t gate = 0;
    const uint32_t drow = dst + static_cast<uint32_t>((row >> 3) * (kUH * 16) + (row & 7) * 16 + half * 8 * 128);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      uint32_t pk[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int c = 8 * q + 2 * e;
        const float v0 = __uint_as_float(c < 32 ? ra[c] : rb[c - 32]) + bias[64 * half + c];
        const float v1 = __uint_as_float(c < 32 ? ra[c + 1] : rb[c - 31]) + bias[64 * half + c + 1];
        gate |= (static_cast<uint64_t>(v0 > 0.0f) << c) | (static_cast<uint64_t>(v1 > 0.0f) << (c + 1));
        pk[e] = relu_pack_bf16(__float_as_uint(v0), __float_as_uint(v1));
      }
      sts_v4(drow + static_cast<uint32_t>(q * 128), pk[0], pk[1], pk[2], pk[3]);
    }
    return gate;
  };
  // backward epilogue: d h (accumulator) gated by the layer's ReLU -> bf16 -> this thread's row of `dst`
  auto bwd_epilogue = [&](uint64_t gate, uint32_t dst) {
    uint32_t ra[32], rb[32];
    tmem_ld32_nowait(tmem + kColAcc + lane_off + 64u * half, ra);
    tmem_ld32_nowait(tmem + kColAcc + lane_off + 64u * half + 32u, rb);
    tmem_ld_wait();
    const uint32_t drow = dst + static_cast<uint32_t>((row >> 3) * (kUH * 16) + (row & 7) * 16 + half * 8 * 128);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      uint32_t pk[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int c = 8 * q + 2 * e;
        const float v0 = ((gate >> c) & 1u) ? __uint_as_float(c < 32 ? ra[c] : rb[c - 32]) : 0.0f;
        const float v1 = ((gate >> (c + 1)) & 1u) ? __uint_as_float(c < 32 ? ra[c + 1] : rb[c - 31]) : 0.0f;
        pk[e] = pack_bf16(v0, v1);
      }
      sts_v4(drow + static_cast<uint32_t>(q * 128), pk[0], pk[1], pk[2], pk[3]);
    }
  };

  for (int i = 0; i < my_tiles && !timed_out; ++i) {
    const long long row0 = tile_of(i) * kUR;
    const int n_valid = static_cast<int>(min(static_cast<long long>(kUR), rows.n - row0));
    const long long my_row = row < n_valid ? real_row(rows, row0 + row) : -1;
    int action = 0;
    float logp_old = 0.0f, adv = 0.0f, v_old = 0.0f, ret = 0.0f;
    if (half == 0) {
      sm.rmap[row] = my_row;
      if (row < n_valid && my_row < 0) atomicExch(status, kStatusBadIndex);
      if (my_row >= 0) {  // used after the heads: the loads are in flight meanwhile
        action = rows.actions[my_row]; logp_old = rows.logp_old[my_row]; adv = rows.adv[my_row];
        v_old = rows.value_old[my_row * rows.vstride]; ret = rows.ret[my_row * rows.vstride];
      }
    }
    const bool bulk = bulk_ok(i);
    if (bulk) { timed_out |= !mbar_wait(bar_stage, ph_stage); ph_stage ^= 1; }
    if (i > 0) { timed_out |= !mbar_wait(bar_end, ph_end); ph_end ^= 1; }  // the previous tile's d W1 has read x
    if (__syncthreads_or(timed_out)) { timed_out = true; if (tid == 0 && bulk) stage_pending = false; break; }
    if (tid == 0 && bulk) stage_pending = false;
    // ---- the tile's rows as bf16 into x: a warp per row, consecutive lanes consecutive features
    {
      constexpr int G = 4;
      for (int g0 = warp; g0 < kUR; g0 += 8 * G) {
        float v[G][3];
#pragma unroll
        for (int g = 0; g < G; ++g) {
          const int r = g0 + 8 * g;
          const long long src = sm.rmap[r];
#pragma unroll
          for (int q = 0; q < 3; ++q) {
            const int k = lane + 32 * q;
            v[g][q] = 0.0f;
            if (k < D && src >= 0) v[g][q] = bulk ? sm.stage[r * D + k] : rows.x[src * D + k];
          }
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
          const int r = g0 + 8 * g;
#pragma unroll
          for (int q = 0; q < 3; ++q) {
            const int k = lane + 32 * q;
            if (k < D) sts_u16(xt + a_offset<kUK1>(r, k), bf16_bits(v[g][q]));
          }
        }
      }
    }
    fence_async_smem();
    __syncthreads();
    const uint32_t keep = i > 0 ? 1u : 0u;  // the weight-gradient accumulators start at the CTA's first tile
    if (tid == 0) {
      if (bulk_ok(i + 1)) { request_stage(i + 1); stage_pending = true; }
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < kUK1 / 16; ++k)
        mma_bf16(tmem + kColAcc, smem_desc(xt + k * 2 * kALbo, kALbo, (kUK1 / 8) * kALbo), desc_k(w1, kUK1, k), instr_desc(kUR, kUH), k > 0);
      mma_commit(bar_mma);
    }
    timed_out |= !mbar_wait(bar_mma, ph_mma); ph_mma ^= 1;
    tc_fence_after();
    const uint64_t gate1 = fwd_epilogue(b1, h1t);
    fence_async_smem(); tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < kUH / 16; ++k) mma_bf16(tmem + kColAcc, desc_k(h1t, kUH, k), desc_k(w2, kUH, k), instr_desc(kUR, kUH), k > 0);
      mma_commit(bar_mma);
    }
    timed_out |= !mbar_wait(bar_mma, ph_mma); ph_mma ^= 1;
    tc_fence_after();
    const uint64_t gate2 = fwd_epilogue(b2, h2t);
    fence_async_smem(); tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < kUH / 16; ++k) mma_bf16(tmem + kColHead, desc_k(h2t, kUH, k), desc_k(wh, kUH, k), instr_desc(kUR, kUHeads), k > 0);
      mma_commit(bar_mma);
    }
    timed_out |= !mbar_wait(bar_mma, ph_mma); ph_mma ^= 1;
    tc_fence_after();
    // ---- loss terms and the per-row derivatives with respect to the six logits and the value (thread = row)
    if (half == 0) {
      float hv[16], d[8];
      tmem_ld16(tmem + kColHead + lane_off, hv);
#pragma unroll
      for (int k = 0; k < 8; ++k) d[k] = 0.0f;
      if (my_row >= 0) {
        float l[kActions], m = -INFINITY, sum = 0.0f;
#pragma unroll
        for (int k = 0; k < kActions; ++k) { l[k] = hv[k] + bh[k]; m = fmaxf(m, l[k]); }
#pragma unroll
        for (int k = 0; k < kActions; ++k) sum += expf(l[k] - m);
        const float lse = m + logf(sum);
        float ent = 0.0f, p[kActions], lp[kActions], lpa = 0.0f;
#pragma unroll
        for (int k = 0; k < kActions; ++k) {
          lp[k] = l[k] - lse; p[k] = expf(lp[k]); ent -= p[k] * lp[k];
          if (k == action) lpa = lp[k];
        }
        const float rho = expf(lpa - logp_old);
        const float ahat = (adv - mean) * inv_std;
        const float clipped = fminf(fmaxf(rho, 1.0f - hp.clip_eps), 1.0f + hp.clip_eps);
        const float s1 = rho * ahat, s2 = clipped * ahat;
        const bool inside = rho >= 1.0f - hp.clip_eps && rho <= 1.0f + hp.clip_eps;
        const float d_logp = (inside || s1 < s2) ? -s1 * inv_n : 0.0f;  // the clipped branch is constant in rho
#pragma unroll
        for (int k = 0; k < kActions; ++k)
          d[k] = d_logp * ((k == action ? 1.0f : 0.0f) - p[k]) + hp.ent_coef * inv_n * p[k] * (lp[k] + ent);
        t_actor += fminf(s1, s2);
        t_ent += ent;
        const float v = hv[kActions] + bh[kActions];
        const float u = v - ret, uc = v_old + fminf(fmaxf(v - v_old, -hp.clip_eps), hp.clip_eps) - ret;
        const bool in_range = fabsf(v - v_old) <= hp.clip_eps;
        d[kActions] = (in_range || u * u > uc * uc) ? hp.vf_coef * u * inv_n : 0.0f;
        t_value += 0.5 * fmaxf(u * u, uc * uc);
      }
      // columns 0..6: the derivatives; column 7: one (it turns the d z^T products into column sums)
      sts_v4(dht + static_cast<uint32_t>((row >> 3) * (kUHeads * 16) + (row & 7) * 16), pack_bf16(d[0], d[1]), pack_bf16(d[2], d[3]),
             pack_bf16(d[4], d[5]), pack_bf16(d[6], 1.0f));
      // the heads' bias gradients sum the unrounded derivatives: over the warp here, over the warps below
#pragma unroll
      for (int k = 0; k <= kActions; ++k) {
        float s = d[k];
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
        if (lane == 0) sm.red[warp][k] = s;
      }
    }
    fence_async_smem(); tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      // d h2 = dhead . Wh (K = the 16 head columns)
      mma_bf16(tmem + kColAcc, desc_k(dht, kUHeads, 0), desc_mn(wh, kUH, 0), instr_desc(kUR, kUH) | kBmn, 0);
      mma_commit(bar_mma);
      // d Wh^T [unit][head column] += h2^T . dhead (K = rows)
#pragma unroll
      for (int k = 0; k < kUR / 16; ++k)
        mma_bf16(tmem + kColDWh, desc_mn(h2t, kUH, k), desc_mn(dht, kUHeads, k), instr_desc(kUH, kUHeads) | kAmn | kBmn, keep | (k > 0));
    }
    if (tid <= kActions) gbh += (sm.red[0][tid] + sm.red[1][tid]) + (sm.red[2][tid] + sm.red[3][tid]);
    timed_out |= !mbar_wait(bar_mma, ph_mma); ph_mma ^= 1;
    tc_fence_after();
    bwd_epilogue(gate2, dz2t);
    fence_async_smem(); tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      // d h1 = d z2 . W2 (K = the out units of layer 2)
#pragma unroll
      for (int k = 0; k < kUH / 16; ++k) mma_bf16(tmem + kColAcc, desc_k(dz2t, kUH, k), desc_mn(w2, kUH, k), instr_desc(kUR, kUH) | kBmn, k > 0);
      mma_commit(bar_mma);
      // d W2 [out][in] += d z2^T . h1 and d b2 [out] += d z2^T . ones (K = rows)
#pragma unroll
      for (int k = 0; k < kUR / 16; ++k)
        mma_bf16(tmem + kColDW2, desc_mn(dz2t, kUH, k), desc_mn(h1t, kUH, k), instr_desc(kUH, kUH) | kAmn | kBmn, keep | (k > 0));
#pragma unroll
      for (int k = 0; k < kUR / 16; ++k)
        mma_bf16(tmem + kColDB2, desc_mn(dz2t, kUH, k), desc_mn(dht, kUHeads, k), instr_desc(kUH, kUHeads) | kAmn | kBmn, keep | (k > 0));
    }
    timed_out |= !mbar_wait(bar_mma, ph_mma); ph_mma ^= 1;  // d h1 is there, and h2's last reader (d Wh) is done
    tc_fence_after();
    bwd_epilogue(gate1, dz1t);
    fence_async_smem(); tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < kUR / 16; ++k)
        mma_bf16(tmem + kColDW1, desc_mn(dz1t, kUH, k), smem_desc(xt + k * 2 * (kUK1 / 8) * kALbo, (kUK1 / 8) * kALbo, kALbo),
                 instr_desc(kUH, kUK1) | kAmn | kBmn, keep | (k > 0));
#pragma unroll
      for (int k = 0; k < kUR / 16; ++k)
        mma_bf16(tmem + kColDB1, desc_mn(dz1t, kUH, k), desc_mn(dht, kUHeads, k), instr_desc(kUH, kUHeads) | kAmn | kBmn, keep | (k > 0));
      mma_commit(bar_end);
    }
    timed_out = __syncthreads_or(timed_out) != 0;
  }
  // ---- the CTA's slice: accumulators out of tensor memory, once
  if (my_tiles > 0 && !timed_out) timed_out |= !mbar_wait(bar_end, ph_end);
  timed_out = __syncthreads_or(timed_out) != 0;
  if (!timed_out && my_tiles > 0) {
    tc_fence_after();
    float *part = partial + static_cast<size_t>(blockIdx.x) * n_params;
    const int unit = (warp & 3) * 32 + lane;  // tensor-memory lane = out unit (d W2, d W1, d b) or hidden unit (d Wh)
    float v[32];
    if (half == 0) {
      for (int c0 = 0; c0 < kUH; c0 += 16) {
        tmem_ld16(tmem + kColDW2 + lane_off + static_cast<uint32_t>(c0), v);
        if (unit < H)
          for (int c = 0; c < 16; ++c)
            if (c0 + c < H) part[off.W2 + static_cast<size_t>(unit) * H + c0 + c] = v[c];
      }
    } else {
      for (int c0 = 0; c0 < kUK1; c0 += 16) {
        tmem_ld16(tmem + kColDW1 + lane_off + static_cast<uint32_t>(c0), v);
        if (unit < H)
          for (int c = 0; c < 16; ++c)
            if (c0 + c < D) part[off.W1 + static_cast<size_t>(unit) * D + c0 + c] = v[c];
      }
      tmem_ld16(tmem + kColDWh + lane_off, v);
      if (unit < H) {
        for (int k = 0; k < kActions; ++k) part[off.Wa + static_cast<size_t>(k) * H + unit] = v[k];
        part[off.Wv + unit] = v[kActions];
      }
      tmem_ld16(tmem + kColDB2 + lane_off, v);
      if (unit < H) part[off.b2 + unit] = v[7];
      tmem_ld16(tmem + kColDB1 + lane_off, v);
      if (unit < H) part[off.b1 + unit] = v[7];
    }
    if (tid < kActions) part[off.ba + tid] = gbh;
    if (tid == kActions) part[off.bv] = gbh;
  }
  {  // loss-term sums of the warp, lane 0 writes them (warps 4..7 hold zeros)
    double s[3] = {t_actor, t_ent, t_value};
#pragma unroll
    for (int k = 0; k < 3; ++k)
      for (int o = 16; o > 0; o >>= 1) s[k] += __shfl_xor_sync(0xFFFFFFFFu, s[k], o);
    if (lane == 0) {
      double *tp = term_partial + (static_cast<size_t>(blockIdx.x) * 8 + warp) * 3;
      tp[0] = s[0]; tp[1] = s[1]; tp[2] = s[2];
    }
  }
  if (timed_out && tid == 0) {
    atomicExch(status, kStatusTimeout);
    if (stage_pending) mbar_wait(bar_stage, ph_stage);  // let the copy in flight land before the block goes away
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

}  // namespace

bool ppo_tc_supported(const mava_config_t &cfg, int D) {
  return cfg.net_kind == MAVA_NET_SHARED_TORSO && cfg.hidden <= kUH && cfg.hidden % 8 == 0 && D <= kUK1;
}

size_t ppo_tc_image_bytes() { return kImgBytes; }

cudaError_t launch_ppo_net_tc(mava_rollout *h, const float *params_dev, const ParamLayout &L, const UpdRows &rows, const UpdHyper &hp,
                              const double *adv_stats, void *image, float *partial, size_t n_params, double *term_partial, int slices) {
  prep_upd_tc_kernel<<<32, 256, 0, h->stream>>>(params_dev, static_cast<unsigned char *>(image), L, h->D, h->cfg.hidden);
  h->launches += 1;
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  const size_t smem = sizeof(UtcSmem);
  err = cudaFuncSetAttribute(ppo_net_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (err != cudaSuccess) return err;
  const Offsets off{L.W1, L.b1, L.W2, L.b2, L.Wa, L.ba, L.Wv, L.bv};
  ppo_net_tc_kernel<<<slices, kUThreads, smem, h->stream>>>(static_cast<const unsigned char *>(image), rows, hp, adv_stats, partial, n_params,
                                                            term_partial, h->d_status, off, h->D, h->cfg.hidden);
  h->launches += 1;
  return cudaGetLastError();
}

}  // namespace mava
