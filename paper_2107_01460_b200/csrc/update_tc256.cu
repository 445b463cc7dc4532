// Update block on the tensor cores for hidden width 256 (sm_100a, tcgen05): the actor / shared-torso net of the two
// largest shapes.  The weight gradient of the second layer alone (256 x 256 fp32) fills all 512 columns of an SM's tensor
// memory, and the weights (184 KB in bf16) leave no room for bf16 activation tiles in shared memory, so the work is cut in
// two kernels that meet in a staging buffer (a chunk of rows at a time, so that the buffer stays small):
//   row kernel     per 128-row tile: forward and backward through the layers with the activations kept in tensor memory
//                  as the A operand of the next product (as the rollout does), the loss and its per-row derivatives in
//                  fp32; every bf16 matrix that a weight gradient needs (x, h1, h2, d z2, d z1, the derivatives of the
//                  heads) is written to the staging buffer as tiles in the canonical core-matrix layout [row][feature];
//   weight kernel  streams those tiles back with bulk copies and reads them with the row index as K (MN-major operands,
//                  see update_tc.cu): d W2 += d z2^T . h1 by one group of CTAs (four 128 x 128 accumulators = all of
//                  tensor memory), d W1 += d z1^T . x and d Wh^T += h2^T . dhead by another; the bias gradients are column
//                  sums of the same tiles by the plain ALUs.  Every CTA adds its accumulators into its own slice of the
//                  partial-gradient array, which update.cu's reducer sums in slice order: same bytes on every call.
// Rounding points are those of the bf16-operand mode of the float64 oracle.  Every mbarrier wait is bounded.
#include <cuda_bf16.h>

#include "common.cuh"
#include "layout.h"
#include "tc_common.cuh"
#include "update_common.cuh"

namespace mava {
namespace {

constexpr int kR = 128;       // rows per tile
constexpr int kH = 256;       // hidden width
constexpr int kK1 = 96;       // input width, padded (D = 81, 85)
constexpr int kHeads = 16;
constexpr int kThreads = 256;

// Image in shared memory: W1 (one input slab) | W2 | Wh | b1 | b2 | bh.  In global memory the image holds all slabs of
// W1 first (kImgW2 bytes each), then the rest in the same order.
constexpr uint32_t kImgW1 = 0, kImgW2 = kImgW1 + kH * kK1 * 2, kImgWh = kImgW2 + kH * kH * 2;
constexpr uint32_t kImgB1 = kImgWh + kHeads * kH * 2, kImgB2 = kImgB1 + kH * 4, kImgBh = kImgB2 + kH * 4;
constexpr uint32_t kImgBytes = kImgBh + 32;
static_assert(kImgBytes % 16 == 0, "bulk copies");

// staging buffer, per tile: one x tile [128][96] per input slab; h1, h2, d z2, d z1 as two unit halves [128][128] each;
// dhead [128][16].  An input slab is one agent's observation: the actor / shared-torso net has one, the centralised
// critic (input = the agents' observations side by side) one per agent.
constexpr uint32_t kXLbo = kALbo, kXSbo = (kK1 / 8) * kALbo;  // x tile: feature chunks 144 bytes apart (the converter's
                                                               // 2-byte stores then spread over the banks), row groups 1728
constexpr size_t kStXBytes = (kR / 8) * kXSbo;
constexpr size_t kHalfBytes = kR * 128 * 2, kActBytes = 2 * kHalfBytes;
constexpr size_t kStDhBytes = kR * kHeads * 2;
struct StageLayout {
  size_t x, h1, h2, dz2, dz1, dh, tile;
};
__host__ __device__ inline StageLayout stage_layout(int slabs) {
  StageLayout L;
  L.x = 0; L.h1 = static_cast<size_t>(slabs) * kStXBytes; L.h2 = L.h1 + kActBytes; L.dz2 = L.h2 + kActBytes; L.dz1 = L.dz2 + kActBytes;
  L.dh = L.dz1 + kActBytes; L.tile = L.dh + kStDhBytes;  // 290 816 bytes with one slab
  return L;
}

constexpr uint32_t kColAcc = 0, kColHid = 256, kColHead = 384, kTmemRow = 512;

struct RowSmem {
  alignas(128) unsigned char img[(kImgBytes + 127) / 128 * 128];
  alignas(128) unsigned char x[kStXBytes];
  alignas(128) unsigned char dhead[kR * kHeads * 2];
  long long rmap[kR];
  float red[4][8];
  alignas(8) uint64_t bar_load, bar_mma, bar_mmb, bar_w1;  // bar_mmb: the second column half of a product issued in halves
  uint32_t tmem_base;
};

// Which net the kernels work on: offsets of its layers in the flat parameter (= gradient) array and its input shape.
struct Net256 {
  size_t W1, b1, W2, b2, Wa, ba, Wv, bv;
  int D;          // width of one input slab (an agent's observation)
  int slabs;      // 1, or the number of agents for the centralised critic
  int w1_ld;      // input width of the first layer = slabs * D
  int has_actor, has_value;
};

__global__ void prep_upd256_kernel(const float *__restrict__ params, unsigned char *__restrict__ image, Net256 net) {
  const int tid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
  const int D = net.D;
  for (int i = tid; i < net.slabs * kH * kK1; i += nth) {
    const int a = i / (kH * kK1), r = i - a * (kH * kK1), n = r / kK1, k = r - n * kK1;
    reinterpret_cast<__nv_bfloat16 *>(image + static_cast<size_t>(a) * kImgW2)[canon_offset(n, k, kK1) / 2] =
        __float2bfloat16_rn(k < D ? params[net.W1 + static_cast<size_t>(n) * net.w1_ld + a * D + k] : 0.0f);
  }
  unsigned char *rest = image + static_cast<size_t>(net.slabs) * kImgW2 - kImgW2;  // so that rest + kImgX is where X lies
  auto bf = [&](uint32_t off) { return reinterpret_cast<__nv_bfloat16 *>(rest + off); };
  for (int i = tid; i < kH * kH; i += nth) {
    const int n = i / kH, k = i - n * kH;
    bf(kImgW2)[canon_offset(n, k, kH) / 2] = __float2bfloat16_rn(params[net.W2 + static_cast<size_t>(n) * kH + k]);
  }
  for (int i = tid; i < kHeads * kH; i += nth) {
    const int n = i / kH, k = i - n * kH;
    float v = 0.0f;
    if (n < kActions && net.has_actor) v = params[net.Wa + static_cast<size_t>(n) * kH + k];
    else if (n == kActions && net.has_value) v = params[net.Wv + k];
    bf(kImgWh)[canon_offset(n, k, kH) / 2] = __float2bfloat16_rn(v);
  }
  float *b1 = reinterpret_cast<float *>(rest + kImgB1), *b2 = reinterpret_cast<float *>(rest + kImgB2), *bh = reinterpret_cast<float *>(rest + kImgBh);
  for (int i = tid; i < kH; i += nth) { b1[i] = params[net.b1 + i]; b2[i] = params[net.b2 + i]; }
  if (tid < 8) bh[tid] = (tid < kActions && net.has_actor) ? params[net.ba + tid] : ((tid == kActions && net.has_value) ? params[net.bv] : 0.0f);
}

__device__ __forceinline__ uint64_t desc_k(uint32_t tile, int C, int k) { return smem_desc(tile + k * 256, 128, C * 16); }
__device__ __forceinline__ uint64_t desc_mn(uint32_t tile, int C, int k) { return smem_desc(tile + k * 2 * C * 16, C * 16, 128); }
constexpr uint32_t kAmn = 1u << 15, kBmn = 1u << 16;

__device__ __forceinline__ uint4 lds_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void stg_v4(void *p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.global.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// ---- row kernel ------------------------------------------------------------------------------------------------------
// Tiles [tile0, tile0 + n_tiles) of the minibatch; tile t's staging record is number t - tile0.
__global__ void __launch_bounds__(kThreads, 1)
ppo_rows256_kernel(const unsigned char *__restrict__ image, UpdRows rows, UpdHyper hp, const double *__restrict__ adv_stats,
                   unsigned char *__restrict__ staging, long long tile0, int n_tiles, float *__restrict__ partial, size_t n_params,
                   double *__restrict__ term_partial, int *status, Net256 net) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  RowSmem &sm = *reinterpret_cast<RowSmem *>(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int row = tid & (kR - 1), half = tid >> 7;
  const uint32_t bar_load = smem_u32(&sm.bar_load), bar_mma = smem_u32(&sm.bar_mma), bar_mmb = smem_u32(&sm.bar_mmb), bar_w1 = smem_u32(&sm.bar_w1);
  const int D = net.D, slabs = net.slabs, has_value = net.has_value, has_actor = net.has_actor;
  const StageLayout SL = stage_layout(slabs);
  const unsigned char *image_rest = image + static_cast<size_t>(slabs) * kImgW2;  // W2 | Wh | biases
  if (tid == 0) {
    mbar_init(bar_load, 1); mbar_init(bar_mma, 1); mbar_init(bar_mmb, 1); mbar_init(bar_w1, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)), "r"(kTmemRow) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  for (int i = tid; i < static_cast<int>(sizeof(sm.x) / 16); i += kThreads) sts_zero16(smem_u32(sm.x) + 16u * i);
  for (int i = tid; i < static_cast<int>(sizeof(sm.dhead) / 16); i += kThreads) sts_zero16(smem_u32(sm.dhead) + 16u * i);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (tid == 0) {  // everything but W1 stays for the whole run; with one slab W1 does too
    constexpr uint32_t kChunk = 16384;
    const uint32_t first = slabs == 1 ? 0u : kImgW2;
    mbar_expect_tx(bar_load, kImgBytes - first);
    for (uint32_t o = first; o < kImgBytes; o += kChunk)
      bulk_load(smem_u32(sm.img + o), (o < kImgW2 ? image : image_rest - kImgW2) + o, min(kChunk, kImgBytes - o), bar_load);
  }
  bool timed_out = !mbar_wait(bar_load, 0);
  timed_out = __syncthreads_or(timed_out) != 0;

  const uint32_t tmem = sm.tmem_base;
  const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
  const uint32_t w1 = smem_u32(sm.img + kImgW1), w2 = smem_u32(sm.img + kImgW2), wh = smem_u32(sm.img + kImgWh);
  const uint32_t xt = smem_u32(sm.x), dht = smem_u32(sm.dhead);
  const float *b1 = reinterpret_cast<const float *>(sm.img + kImgB1), *b2 = reinterpret_cast<const float *>(sm.img + kImgB2),
              *bh = reinterpret_cast<const float *>(sm.img + kImgBh);
  const float mean = static_cast<float>(adv_stats[0]);
  const float inv_std = 1.0f / (static_cast<float>(adv_stats[1]) + 1e-8f);
  const float inv_n = 1.0f / static_cast<float>(rows.n);
  const int my_tiles = static_cast<int>(blockIdx.x) < n_tiles ? (n_tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x) : 0;

  uint32_t ph = 0, phb = 0, ph_w1 = 0;
  double t_actor = 0.0, t_ent = 0.0, t_value = 0.0;
  float gbh = 0.0f;
  // this thread's 16-byte pieces of a staged activation: unit half `half`, its own row
  // a staged activation tile is [128 rows][256 units] in the canonical layout: 8-row groups 4096 bytes apart, a row's
  // 16-byte pieces (8 units) 128 bytes apart; this thread's units start at piece 16 * half
  const size_t act_row_off = static_cast<size_t>((row >> 3) * 4096 + (row & 7) * 16) + static_cast<size_t>(half) * 2048;

  // 128 accumulator columns of this thread (+ bias, ReLU) -> bf16 -> tensor memory (A operand of the next product) and
  // the staged tile; gate bits out
  // (the load of the next 32 columns is in flight while the current 32 are converted; biases come in as 16-byte reads)
  auto fwd_batch = [&](const uint32_t *ra, const float *bias, int c0, unsigned char *stage_act, uint32_t &g_out) {
    uint32_t pk[16], g = 0;
#pragma unroll
    for (int e4 = 0; e4 < 8; ++e4) {
      const float4 b = *reinterpret_cast<const float4 *>(bias + 128 * half + c0 + 4 * e4);
      const float v0 = __uint_as_float(ra[4 * e4]) + b.x, v1 = __uint_as_float(ra[4 * e4 + 1]) + b.y;
      const float v2 = __uint_as_float(ra[4 * e4 + 2]) + b.z, v3 = __uint_as_float(ra[4 * e4 + 3]) + b.w;
      g |= (static_cast<uint32_t>(v0 > 0.0f) << (4 * e4)) | (static_cast<uint32_t>(v1 > 0.0f) << (4 * e4 + 1)) |
           (static_cast<uint32_t>(v2 > 0.0f) << (4 * e4 + 2)) | (static_cast<uint32_t>(v3 > 0.0f) << (4 * e4 + 3));
      pk[2 * e4] = relu_pack_bf16(__float_as_uint(v0), __float_as_uint(v1));
      pk[2 * e4 + 1] = relu_pack_bf16(__float_as_uint(v2), __float_as_uint(v3));
    }
    g_out = g;
    tmem_st16(tmem + kColHid + lane_off + static_cast<uint32_t>((128 * half + c0) / 2), pk);
#pragma unroll
    for (int q = 0; q < 4; ++q)
      stg_v4(stage_act + act_row_off + static_cast<size_t>((c0 / 8 + q) * 128), pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
  };
  auto fwd_epilogue = [&](const float *bias, unsigned char *stage_act, uint32_t gate[4]) {
    uint32_t ra[32], rb[32];
    const uint32_t acc = tmem + kColAcc + lane_off + 128u * half;
    tmem_ld32_nowait(acc, ra);
#pragma unroll 1
    for (int c0 = 0; c0 < 128; c0 += 64) {
      tmem_ld_wait(); tmem_ld32_nowait(acc + static_cast<uint32_t>(c0 + 32), rb); fwd_batch(ra, bias, c0, stage_act, gate[c0 / 32]);
      tmem_ld_wait();
      if (c0 == 0) tmem_ld32_nowait(acc + 64u, ra);
      fwd_batch(rb, bias, c0 + 32, stage_act, gate[c0 / 32 + 1]);
    }
    tmem_st_wait();
  };
  auto bwd_batch = [&](const uint32_t *ra, uint32_t g, int c0, unsigned char *stage_act, bool to_tmem) {
    uint32_t pk[16];
#pragma unroll
    for (int e = 0; e < 16; ++e)
      pk[e] = pack_bf16(((g >> (2 * e)) & 1u) ? __uint_as_float(ra[2 * e]) : 0.0f, ((g >> (2 * e + 1)) & 1u) ? __uint_as_float(ra[2 * e + 1]) : 0.0f);
    if (to_tmem) tmem_st16(tmem + kColHid + lane_off + static_cast<uint32_t>((128 * half + c0) / 2), pk);
#pragma unroll
    for (int q = 0; q < 4; ++q)
      stg_v4(stage_act + act_row_off + static_cast<size_t>((c0 / 8 + q) * 128), pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
  };
  auto bwd_epilogue = [&](const uint32_t gate[4], unsigned char *stage_act, bool to_tmem) {
    uint32_t ra[32], rb[32];
    const uint32_t acc = tmem + kColAcc + lane_off + 128u * half;
    tmem_ld32_nowait(acc, ra);
#pragma unroll 1
    for (int c0 = 0; c0 < 128; c0 += 64) {
      tmem_ld_wait(); tmem_ld32_nowait(acc + static_cast<uint32_t>(c0 + 32), rb); bwd_batch(ra, gate[c0 / 32], c0, stage_act, to_tmem);
      tmem_ld_wait();
      if (c0 == 0) tmem_ld32_nowait(acc + 64u, ra);
      bwd_batch(rb, gate[c0 / 32 + 1], c0 + 32, stage_act, to_tmem);
    }
    if (to_tmem) tmem_st_wait();
  };

  for (int i = 0; i < my_tiles && !timed_out; ++i) {
    const int lt = static_cast<int>(blockIdx.x) + i * static_cast<int>(gridDim.x);  // tile inside the chunk
    const long long row0 = (tile0 + lt) * kR;
    unsigned char *st = staging + static_cast<size_t>(lt) * SL.tile;
    const int n_valid = static_cast<int>(min(static_cast<long long>(kR), rows.n - row0));
    const long long my_row = row < n_valid ? real_row(rows, row0 + row) : -1;
    int action = 0;
    float logp_old = 0.0f, adv = 0.0f, v_old = 0.0f, ret = 0.0f;
    if (half == 0) {
      sm.rmap[row] = my_row;
      if (row < n_valid && my_row < 0) atomicExch(status, kStatusBadIndex);
      if (my_row >= 0) {
        if (has_actor) { action = rows.actions[my_row]; logp_old = rows.logp_old[my_row]; adv = rows.adv[my_row]; }
        if (has_value) { v_old = rows.value_old[my_row * rows.vstride]; ret = rows.ret[my_row * rows.vstride]; }
      }
    }
    // ---- layer 1, one input slab at a time: z1 = sum over slabs of x_a . W1_a^T
    for (int a = 0; a < slabs; ++a) {
      if (a > 0) {  // the previous slab's MMAs (both column halves) have read the x tile and the W1 slab
        timed_out |= !mbar_wait(bar_mma, ph); ph ^= 1;
        timed_out |= !mbar_wait(bar_mmb, phb); phb ^= 1;
      }
      if (tid == 0) {
        bulk_store_wait_read();  // the copies of the x tile (and of the previous tile's dhead tile) have read them
        if (slabs > 1) {         // this slab of W1 comes in while the rows are converted
          mbar_expect_tx(bar_w1, kImgW2);
          for (uint32_t o = 0; o < kImgW2; o += 16384)
            bulk_load(smem_u32(sm.img + o), image + static_cast<size_t>(a) * kImgW2 + o, 16384, bar_w1);
        }
        // the next tile's rows on their way into L2 (a full tile of consecutive rows is one 16-byte aligned block)
        if (a == 0 && rows.env_ids == nullptr && i + 1 < my_tiles && (tile0 + lt + static_cast<long long>(gridDim.x) + 1) * kR <= rows.n)
          asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(rows.x + static_cast<size_t>(tile0 + lt + gridDim.x) * kR * net.w1_ld),
                       "r"(static_cast<uint32_t>(kR * net.w1_ld * 4))
                       : "memory");
      }
      tc_fence_before();
      __syncthreads();
      // the tile's rows (slab a of each) as bf16 into x: a warp per row, consecutive lanes consecutive features
      {
        constexpr int G = 16;  // all of a warp's rows at once: one round trip to L2
        for (int g0 = warp; g0 < kR; g0 += 8 * G) {
          float v[G][3];
#pragma unroll
          for (int g = 0; g < G; ++g) {
            const long long src = sm.rmap[g0 + 8 * g];
#pragma unroll
            for (int q = 0; q < 3; ++q) {
              const int k = lane + 32 * q;
              v[g][q] = (k < D && src >= 0) ? rows.x[src * net.w1_ld + a * D + k] : 0.0f;
            }
          }
#pragma unroll
          for (int g = 0; g < G; ++g)
#pragma unroll
            for (int q = 0; q < 3; ++q) {
              const int k = lane + 32 * q;
              if (k < D) sts_u16(xt + a_offset<kK1>(g0 + 8 * g, k), bf16_bits(v[g][q]));
            }
        }
      }
      fence_async_smem();
      __syncthreads();
      if (tid == 0) {
        bulk_store(st + SL.x + static_cast<size_t>(a) * kStXBytes, xt, static_cast<uint32_t>(kStXBytes));
        if (slabs > 1) { timed_out |= !mbar_wait(bar_w1, ph_w1); ph_w1 ^= 1; }
        tc_fence_after();
#pragma unroll
        // the product in two column halves with a commit each: a thread's epilogue needs its own half only
#pragma unroll
        for (int nh = 0; nh < 2; ++nh) {
#pragma unroll
          for (int k = 0; k < kK1 / 16; ++k)
            mma_bf16(tmem + kColAcc + 128u * nh, smem_desc(xt + k * 2 * kXLbo, kXLbo, kXSbo), desc_k(w1 + nh * 16 * (kK1 * 16), kK1, k),
                     instr_desc(kR, kH / 2), (a > 0) | (k > 0));
          mma_commit(nh == 0 ? bar_mma : bar_mmb);
        }
      }
    }
    if (half == 0) { timed_out |= !mbar_wait(bar_mma, ph); } else { timed_out |= !mbar_wait(bar_mmb, phb); }
    ph ^= 1; phb ^= 1;
    tc_fence_after();
    uint32_t gate1[4], gate2[4];
    fwd_epilogue(b1, st + SL.h1, gate1);
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < kH / 16; ++k) mma_bf16_ts(tmem + kColAcc, tmem + kColHid + k * 8, desc_k(w2, kH, k), instr_desc(kR, kH), k > 0);
      mma_commit(bar_mma);
    }
    timed_out |= !mbar_wait(bar_mma, ph); ph ^= 1;
    tc_fence_after();
    fwd_epilogue(b2, st + SL.h2, gate2);
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < kH / 16; ++k) mma_bf16_ts(tmem + kColHead, tmem + kColHid + k * 8, desc_k(wh, kH, k), instr_desc(kR, kHeads), k > 0);
      mma_commit(bar_mma);
    }
    timed_out |= !mbar_wait(bar_mma, ph); ph ^= 1;
    tc_fence_after();
    if (half == 0) {
      float hv[16], d[8];
      tmem_ld16(tmem + kColHead + lane_off, hv);
#pragma unroll
      for (int k = 0; k < 8; ++k) d[k] = 0.0f;
      if (my_row >= 0 && has_actor) {
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
        const float d_logp = (inside || s1 < s2) ? -s1 * inv_n : 0.0f;
#pragma unroll
        for (int k = 0; k < kActions; ++k)
          d[k] = d_logp * ((k == action ? 1.0f : 0.0f) - p[k]) + hp.ent_coef * inv_n * p[k] * (lp[k] + ent);
        t_actor += fminf(s1, s2);
        t_ent += ent;
      }
      if (my_row >= 0 && has_value) {
        {
          const float v = hv[kActions] + bh[kActions];
          const float u = v - ret, uc = v_old + fminf(fmaxf(v - v_old, -hp.clip_eps), hp.clip_eps) - ret;
          const bool in_range = fabsf(v - v_old) <= hp.clip_eps;
          d[kActions] = (in_range || u * u > uc * uc) ? hp.vf_coef * u * inv_n : 0.0f;
          t_value += 0.5 * fmaxf(u * u, uc * uc);
        }
      }
      sts_v4(dht + static_cast<uint32_t>((row >> 3) * (kHeads * 16) + (row & 7) * 16), pack_bf16(d[0], d[1]), pack_bf16(d[2], d[3]),
             pack_bf16(d[4], d[5]), pack_bf16(d[6], 0.0f));
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
      bulk_store(st + SL.dh, dht, static_cast<uint32_t>(kStDhBytes));
      tc_fence_after();
      mma_bf16(tmem + kColAcc, desc_k(dht, kHeads, 0), desc_mn(wh, kH, 0), instr_desc(kR, kH) | kBmn, 0);  // d h2 = dhead . Wh
      mma_commit(bar_mma);
    }
    if (tid <= kActions) gbh += (sm.red[0][tid] + sm.red[1][tid]) + (sm.red[2][tid] + sm.red[3][tid]);
    timed_out |= !mbar_wait(bar_mma, ph); ph ^= 1;
    tc_fence_after();
    bwd_epilogue(gate2, st + SL.dz2, true);
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
#pragma unroll
      for (int nh = 0; nh < 2; ++nh) {  // d h1 = d z2 . W2, again in two column halves
#pragma unroll
        for (int k = 0; k < kH / 16; ++k)
          mma_bf16_ts(tmem + kColAcc + 128u * nh, tmem + kColHid + k * 8, desc_mn(w2 + nh * 16 * 128, kH, k), instr_desc(kR, kH / 2) | kBmn, k > 0);
        mma_commit(nh == 0 ? bar_mma : bar_mmb);
      }
    }
    if (half == 0) { timed_out |= !mbar_wait(bar_mma, ph); } else { timed_out |= !mbar_wait(bar_mmb, phb); }
    ph ^= 1; phb ^= 1;
    tc_fence_after();
    bwd_epilogue(gate1, st + SL.dz1, false);
    timed_out = __syncthreads_or(timed_out) != 0;
  }
  if (!timed_out) {
    float *part = partial + static_cast<size_t>(blockIdx.x) * n_params;
    if (tid < kActions && has_actor) part[net.ba + tid] += gbh;
    if (tid == kActions && has_value) part[net.bv] += gbh;
  }
  {
    double s[3] = {t_actor, t_ent, t_value};
#pragma unroll
    for (int k = 0; k < 3; ++k)
      for (int o = 16; o > 0; o >>= 1) s[k] += __shfl_xor_sync(0xFFFFFFFFu, s[k], o);
    if (lane == 0) {
      double *tp = term_partial + (static_cast<size_t>(blockIdx.x) * 8 + warp) * 3;
      tp[0] += s[0]; tp[1] += s[1]; tp[2] += s[2];
    }
  }
  if (tid == 0) {
    if (timed_out) atomicExch(status, kStatusTimeout);
    bulk_store_wait_all();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemRow) : "memory");
  }
}

// ---- weight kernel ---------------------------------------------------------------------------------------------------
// CTAs [0, n_w2) sum d W2 and d b2; the others d W1 (one input slab each; CTA index modulo the slab count picks the
// slab), and those of slab 0 also d b1 and d Wh.  A CTA's work items are 32-row pieces of the tiles it owns; an item's operands come in by bulk copies into a ring of stages.  Roles inside the CTA, connected by mbarriers
// only: one producer thread (copies), one MMA thread, eight consumer warps (thread j sums column j of the d z tile for
// the bias gradient).  A stage is free again when its MMAs have completed and every consumer warp has let go of it.
constexpr int kItemRows = 32;
constexpr int kItemsPerTile = kR / kItemRows;
constexpr uint32_t kQ = kItemRows * 128 * 2;                  // half of an item's rows of a [128][256] tile: 8 KB
constexpr uint32_t kW2Stage = 4 * kQ, kW2Stages = 6;          // d z2, h1 (16 KB each: 32 rows x 256 units)
constexpr uint32_t kXPart = (kItemRows / 8) * kXSbo, kDhPart = kItemRows * kHeads * 2;
constexpr uint32_t kW1Stage = 4 * kQ + kXPart + kDhPart, kW1Stages = 5;  // d z1, h2 (16 KB each), x, dhead
constexpr uint32_t kRingBytes = kW2Stage * kW2Stages > kW1Stage * kW1Stages ? kW2Stage * kW2Stages : kW1Stage * kW1Stages;
constexpr int kMaxStages = 6;
constexpr int kWgtThreads = 320, kConsumerWarps = 8;

struct WgtSmem {
  alignas(128) unsigned char ring[kRingBytes];
  alignas(8) uint64_t full[kMaxStages], empty[kMaxStages], done;
  uint32_t tmem_base;
};

__global__ void __launch_bounds__(kWgtThreads, 1)
ppo_weights256_kernel(const unsigned char *__restrict__ staging, int n_tiles, int n_w2, float *__restrict__ partial, size_t n_params,
                      int *status, Net256 net) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  WgtSmem &sm = *reinterpret_cast<WgtSmem *>(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool role_w2 = static_cast<int>(blockIdx.x) < n_w2;
  const int D = net.D, slabs = net.slabs, has_value = net.has_value, has_actor = net.has_actor;
  const StageLayout SL = stage_layout(slabs);
  const int rest = static_cast<int>(gridDim.x) - n_w2;                                  // CTAs of the d W1 group
  const int slab = role_w2 ? 0 : (static_cast<int>(blockIdx.x) - n_w2) % slabs;          // input slab of this CTA
  const int rank = role_w2 ? static_cast<int>(blockIdx.x) : (static_cast<int>(blockIdx.x) - n_w2) / slabs;
  const int peers = role_w2 ? n_w2 : rest / slabs + (slab < rest % slabs ? 1 : 0);
  const bool heads_too = !role_w2 && slab == 0;                                          // d Wh and d b1 ride with slab 0
  const int S = role_w2 ? kW2Stages : kW1Stages;
  const uint32_t stage_bytes = role_w2 ? kW2Stage : kW1Stage;
  const uint32_t ring = smem_u32(sm.ring), full0 = smem_u32(&sm.full[0]), empty0 = smem_u32(&sm.empty[0]), done_bar = smem_u32(&sm.done);
  constexpr uint32_t kCols = 512;
  if (tid == 0) {
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(full0 + 8u * s, 1);
      mbar_init(empty0 + 8u * s, 1 + kConsumerWarps);  // the MMAs' commit and every consumer warp
    }
    mbar_init(done_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)), "r"(kCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  const int my_tiles = rank < n_tiles ? (n_tiles - rank + peers - 1) / peers : 0;
  const int n_items = kItemsPerTile * my_tiles;
  bool timed_out = false;
  float db0 = 0.0f, db1 = 0.0f;  // consumer thread: bias gradient (d b2 or d b1) of its two units over its half of the rows

  if (warp == kConsumerWarps) {
    // ---- producer
    if (lane == 0) {
      int issued = 0;
      for (int u = 0; u < n_items && !timed_out; ++u) {
        const int s = u % S;
        if (u >= S) timed_out |= !mbar_wait(empty0 + 8u * s, ((u / S) - 1) & 1);
        if (timed_out) break;
        // the chunk's last tiles first: the row kernel wrote them last, so they are the ones still in L2
        const int lt = n_tiles - 1 - (rank + (u / kItemsPerTile) * peers), q = u % kItemsPerTile;
        const unsigned char *st = staging + static_cast<size_t>(lt) * SL.tile;
        const uint32_t dst = ring + static_cast<uint32_t>(s) * stage_bytes, bar = full0 + 8u * s;
        mbar_expect_tx(bar, stage_bytes);
        const size_t a = role_w2 ? SL.dz2 : SL.dz1, b = role_w2 ? SL.h1 : SL.h2;
        // an item's 32 rows of a staged tile are four 8-row groups = 16 KB in one piece (two copies of 8 KB each)
        bulk_load(dst, st + a + static_cast<size_t>(q) * 2 * kQ, kQ, bar);
        bulk_load(dst + kQ, st + a + static_cast<size_t>(q) * 2 * kQ + kQ, kQ, bar);
        bulk_load(dst + 2 * kQ, st + b + static_cast<size_t>(q) * 2 * kQ, kQ, bar);
        bulk_load(dst + 3 * kQ, st + b + static_cast<size_t>(q) * 2 * kQ + kQ, kQ, bar);
        if (!role_w2) {
          bulk_load(dst + 4 * kQ, st + SL.x + static_cast<size_t>(slab) * kStXBytes + static_cast<size_t>(q) * kXPart, kXPart, bar);
          bulk_load(dst + 4 * kQ + kXPart, st + SL.dh + static_cast<size_t>(q) * kDhPart, kDhPart, bar);
        }
        issued = u + 1;
      }
      if (timed_out)  // let the copies still in flight land before the block goes away
        for (int u = issued > S ? issued - S : 0; u < issued; ++u) mbar_wait(full0 + 8u * (u % S), (u / S) & 1);
    }
  } else if (warp == kConsumerWarps + 1) {
    // ---- MMA issue
    if (lane == 0) {
      for (int u = 0; u < n_items && !timed_out; ++u) {
        const int s = u % S;
        const uint32_t base = ring + static_cast<uint32_t>(s) * stage_bytes;
        timed_out |= !mbar_wait(full0 + 8u * s, (u / S) & 1);
        if (timed_out) break;
        tc_fence_after();
        const uint32_t keep = u > 0 ? 1u : 0u;
        if (role_w2) {  // d W2 [out half a][all 256 in] += d z2[:, a]^T . h1 over the item's rows: each operand piece is
                        // read from shared memory 1.5 times per product instead of twice with four 128 x 128 products
#pragma unroll
          for (int k = 0; k < kItemRows / 16; ++k)
#pragma unroll
            for (int a = 0; a < 2; ++a)
              mma_bf16(tmem + static_cast<uint32_t>(a * 256), desc_mn(base + a * 2048, 256, k), desc_mn(base + 2 * kQ, 256, k),
                       instr_desc(128, 256) | kAmn | kBmn, keep | (k > 0));
        } else {        // d W1 [out half a][in] += d z1[:, a]^T . x;  d Wh^T [unit half a][head] += h2[:, a]^T . dhead
#pragma unroll
          for (int k = 0; k < kItemRows / 16; ++k)
#pragma unroll
            for (int a = 0; a < 2; ++a) {
              mma_bf16(tmem + static_cast<uint32_t>(a * kK1), desc_mn(base + a * 2048, 256, k), smem_desc(base + 4 * kQ + k * 2 * kXSbo, kXSbo, kXLbo),
                       instr_desc(128, kK1) | kAmn | kBmn, keep | (k > 0));
              if (heads_too)
                mma_bf16(tmem + static_cast<uint32_t>(192 + a * 32), desc_mn(base + 2 * kQ + a * 2048, 256, k), desc_mn(base + 4 * kQ + kXPart, kHeads, k),
                         instr_desc(128, kHeads) | kAmn | kBmn, keep | (k > 0));
            }
        }
        mma_commit(empty0 + 8u * s);  // the stage is free once these MMAs have read it
      }
      if (!timed_out && n_items > 0) mma_commit(done_bar);  // covers every MMA issued above
    }
  } else {
    // ---- consumers: column sums of the d z tile for the bias gradient.  Thread (w, l): units 2p, 2p + 1 with
    // p = 32 (w & 3) + l, over the item's rows 16 (w >> 2) .. + 15, by 4-byte loads.  A warp's 32 unit pairs are eight
    // 16-byte pieces 128 bytes apart, i.e. on the same four banks: each piece's four lanes therefore start at a
    // different row of the 8-row group (row offset 16 bytes = four banks) and a load touches all 32 banks once.  The
    // two row halves are added at the end, in a fixed order: the same bytes on every call.
    const int p = (warp & 3) * 32 + lane;
    const uint32_t my_col = static_cast<uint32_t>((p >> 2) * 128 + (p & 3) * 4) + static_cast<uint32_t>(warp >> 2) * 2 * 4096;
    const int rot = lane >> 2;
    for (int u = 0; u < n_items && !timed_out; ++u) {
      const int s = u % S;
      const uint32_t base = ring + static_cast<uint32_t>(s) * stage_bytes;
      timed_out |= !mbar_wait(full0 + 8u * s, (u / S) & 1);
      if (__any_sync(0xFFFFFFFFu, timed_out)) { timed_out = true; break; }
#pragma unroll
      for (int rg = 0; rg < 2; ++rg)
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint32_t w2 = lds_u32(base + my_col + static_cast<uint32_t>(rg * 4096) + static_cast<uint32_t>(((j + rot) & 7) * 16));
          db0 += __uint_as_float(w2 << 16);
          db1 += __uint_as_float(w2 & 0xFFFF0000u);
        }
      // the stage's next writer is a bulk copy (async proxy); these were generic-proxy reads.  Without the proxy fence
      // the copy may land before the reads have been performed (seen on the GPU as bias sums that changed from call to call).
      fence_async_smem();
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty0 + 8u * s) : "memory");
    }
  }
  // the consumer warps read the accumulators below; the other two warps go straight to the block-wide barrier
  if (warp < kConsumerWarps && n_items > 0 && !timed_out) timed_out |= !mbar_wait(done_bar, 0);
  timed_out = __syncthreads_or(timed_out) != 0;
  {  // the two row halves of the bias sums meet in the ring, which is idle: every copy and every MMA has completed
    float *xch = reinterpret_cast<float *>(sm.ring);
    const int p = (warp & 3) * 32 + lane;
    if (!timed_out && warp >= 4 && warp < kConsumerWarps) { xch[2 * p] = db0; xch[2 * p + 1] = db1; }
    __syncthreads();
    if (!timed_out && warp < 4) { db0 += xch[2 * p]; db1 += xch[2 * p + 1]; }
  }
  if (!timed_out && my_tiles > 0 && warp < kConsumerWarps) {
    tc_fence_after();
    float *part = partial + static_cast<size_t>(blockIdx.x) * n_params;
    const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const int a = warp >> 2, unit = a * 128 + (warp & 3) * 32 + lane;  // out-unit half a; tensor-memory lane = unit inside the half
    float v[16];
    if (role_w2) {
      for (int b = 0; b < 2; ++b)
        for (int c0 = 0; c0 < 128; c0 += 16) {
          tmem_ld16(tmem + lane_off + static_cast<uint32_t>((a * 2 + b) * 128 + c0), v);
          float *dst = part + net.W2 + static_cast<size_t>(unit) * kH + b * 128 + c0;
#pragma unroll
          for (int c = 0; c < 16; ++c) dst[c] += v[c];
        }
      if (warp < 4) { part[net.b2 + 2 * tid] += db0; part[net.b2 + 2 * tid + 1] += db1; }
    } else {
      for (int c0 = 0; c0 < kK1; c0 += 16) {
        tmem_ld16(tmem + lane_off + static_cast<uint32_t>(a * kK1 + c0), v);
        for (int c = 0; c < 16; ++c)
          if (c0 + c < D) part[net.W1 + static_cast<size_t>(unit) * net.w1_ld + slab * D + c0 + c] += v[c];
      }
      if (heads_too) {
        tmem_ld16(tmem + lane_off + static_cast<uint32_t>(192 + a * 32), v);
        if (has_actor)
          for (int k = 0; k < kActions; ++k) part[net.Wa + static_cast<size_t>(k) * kH + unit] += v[k];
        if (has_value) part[net.Wv + unit] += v[kActions];
        if (warp < 4) { part[net.b1 + 2 * tid] += db0; part[net.b1 + 2 * tid + 1] += db1; }
      }
    }
  }
  if (timed_out && tid == 0) atomicExch(status, kStatusTimeout);
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kCols) : "memory");
  }
}

}  // namespace

bool ppo_tc256_supported(const mava_config_t &cfg, int D) { return cfg.hidden == kH && D <= kK1 && D > 64; }
size_t ppo_tc256_image_bytes(int slabs) { return static_cast<size_t>(slabs - 1) * kImgW2 + kImgBytes; }
size_t ppo_tc256_staging_bytes(int chunk_tiles, int slabs) { return static_cast<size_t>(chunk_tiles) * stage_layout(slabs).tile; }

cudaError_t launch_ppo_net_tc256(mava_rollout *h, const float *params_dev, const Tc256Net &desc, const UpdRows &rows, const UpdHyper &hp,
                                 const double *adv_stats, void *image, void *staging, int chunk_tiles, float *partial, size_t n_params,
                                 double *term_partial, int slices) {
  Net256 net{};
  net.W1 = desc.W1; net.b1 = desc.b1; net.W2 = desc.W2; net.b2 = desc.b2; net.Wa = desc.Wa; net.ba = desc.ba; net.Wv = desc.Wv; net.bv = desc.bv;
  net.D = h->D; net.slabs = desc.slabs; net.w1_ld = desc.slabs * h->D; net.has_actor = desc.has_actor ? 1 : 0; net.has_value = desc.has_value ? 1 : 0;
  prep_upd256_kernel<<<64, 256, 0, h->stream>>>(params_dev, static_cast<unsigned char *>(image), net);
  h->launches += 1;
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  err = cudaFuncSetAttribute(ppo_rows256_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(sizeof(RowSmem)));
  if (err == cudaSuccess)
    err = cudaFuncSetAttribute(ppo_weights256_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(sizeof(WgtSmem)));
  if (err != cudaSuccess) return err;
  const long long tiles = (rows.n + kR - 1) / kR;
  // CTAs of the weight kernel by the bytes each group streams per tile: 128 KB for d W2 against 156 KB per input slab
  int n_w2 = (slices * 128 + (128 + 156 * net.slabs) / 2) / (128 + 156 * net.slabs);
  if (n_w2 < 1) n_w2 = 1;
  if (slices - n_w2 < net.slabs) return cudaErrorInvalidConfiguration;  // every slab needs a CTA
  for (long long t0 = 0; t0 < tiles; t0 += chunk_tiles) {
    const int nt = static_cast<int>(tiles - t0 < chunk_tiles ? tiles - t0 : chunk_tiles);
    ppo_rows256_kernel<<<slices, kThreads, sizeof(RowSmem), h->stream>>>(static_cast<const unsigned char *>(image), rows, hp, adv_stats,
                                                                         static_cast<unsigned char *>(staging), t0, nt, partial, n_params,
                                                                         term_partial, h->d_status, net);
    ppo_weights256_kernel<<<slices, kWgtThreads, sizeof(WgtSmem), h->stream>>>(static_cast<const unsigned char *>(staging), nt, n_w2, partial,
                                                                               n_params, h->d_status, net);
    h->launches += 2;
  }
  return cudaGetLastError();
}

}  // namespace mava
