// Centralised critic (MAPPO) on the tensor cores, as two batched kernels over the stored
// trajectory: the critic's value does not feed the next environment step, so it is taken off the
// rollout's serial chain and computed for all (T+1)*E environment-steps at once.
//   layer-1 kernel: h1 = relu(X C1^T + c1), X = the N observations of an environment-step
//     concatenated (N*D fp32, contiguous in the time-major obs array).  C1 (bf16, canonical K-major
//     layout) stays in shared memory; producer warps stream the 128-row tiles through a ring of
//     48-column A buffers (fp32 -> bf16 on the way in), one thread issues the MMAs, epilogue warps
//     leave h1 as bf16 tiles, already in the operand layout, in a scratch array.
//   layer-2 kernel: v = Cv relu(h1 C2^T + c2) + cv.  C2 stays in shared memory, the h1 tiles come
//     in by bulk copies; two thread groups alternate tiles, one in its epilogue (ReLU, bf16
//     rounding, dot product with Cv) while the other's MMAs run.  The value is written to the N
//     slots of its environment-step.
// Every mbarrier wait is bounded; a group that gives up records kStatusTimeout and leaves.
#include <cuda.h>  // CUtensorMap and its enums (types only: nothing of the driver library is linked)

#include "common.cuh"
#include "layout.h"
#include "tc_common.cuh"

namespace mava {
namespace {

constexpr int kCH = 256;  // hidden width of the compiled critic

template <int N>
struct CriticShape {
  static constexpr int D = kObsFixed + N;
  static constexpr int KJ = N * D;                        // joint observation width
  static constexpr int K1 = (KJ + 2 + 15) / 16 * 16;      // + two ones columns that carry c1
  static constexpr int CHUNK = 48;                        // K columns per A buffer (3 MMA K steps)
  static constexpr int NCHUNK = K1 / CHUNK;
  static_assert(K1 % CHUNK == 0 && KJ % 4 == 0, "chunking assumes float4 rows and whole chunks");
  static constexpr uint32_t C1_BYTES = kCH * K1 * 2;
  // A buffers of layer 1: core matrices of a row group 144 bytes apart, so that the twelve 8-byte
  // stores a row gets from consecutive threads fall into different banks
  static constexpr uint32_t A_LBO = 144;
  static constexpr uint32_t A_SBO = (CHUNK / 8) * A_LBO;
  static constexpr uint32_t A_BUF_BYTES = (kTileRows / 8) * A_SBO;
  // layer-2 image: C2 | c2 bias tile | ones tile | Cv (bf16-rounded, as fp32) | cv
  static constexpr uint32_t C2_OFF = 0, C2_BYTES = kCH * kCH * 2;
  static constexpr uint32_t B2_OFF = C2_OFF + C2_BYTES, B2_BYTES = kCH * 16 * 2;
  static constexpr uint32_t ONES_OFF = B2_OFF + B2_BYTES, ONES_BYTES = kTileRows * 16 * 2;
  static constexpr uint32_t CV_OFF = ONES_OFF + ONES_BYTES, CV_BYTES = kCH * 4 + 16;
  static constexpr uint32_t L2_BYTES = CV_OFF + CV_BYTES;
  static constexpr uint32_t H1_TILE_BYTES = kTileRows * kCH * 2;
  static constexpr uint32_t IMAGE_BYTES = C1_BYTES + L2_BYTES;
};

template <int N>
__global__ void prep_critic_kernel(const float *__restrict__ params, unsigned char *__restrict__ image, ParamLayout L) {
  using S = CriticShape<N>;
  constexpr int KJ = S::KJ, K1 = S::K1;
  auto at = [&](uint32_t off) { return reinterpret_cast<__nv_bfloat16 *>(image + off); };
  const int tid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
  for (int i = tid; i < kCH * K1; i += nth) {
    const int n = i / K1, k = i - n * K1;
    __nv_bfloat16 v = __float2bfloat16_rn(k < KJ ? params[L.C1 + static_cast<size_t>(n) * KJ + k] : 0.0f);
    if (k == KJ || k == KJ + 1) {
      __nv_bfloat16 hi, lo;
      split_bf16(params[L.c1 + n], hi, lo);
      v = (k == KJ) ? hi : lo;
    }
    at(0)[canon_offset(n, k, K1) / 2] = v;
  }
  unsigned char *l2 = image + S::C1_BYTES;
  auto at2 = [&](uint32_t off) { return reinterpret_cast<__nv_bfloat16 *>(l2 + off); };
  for (int i = tid; i < kCH * kCH; i += nth) {
    const int n = i / kCH, k = i - n * kCH;
    at2(S::C2_OFF)[canon_offset(n, k, kCH) / 2] = __float2bfloat16_rn(params[L.C2 + static_cast<size_t>(n) * kCH + k]);
  }
  for (int i = tid; i < kCH * 16; i += nth) {
    const int n = i / 16, k = i - n * 16;
    __nv_bfloat16 hi, lo;
    split_bf16(params[L.c2 + n], hi, lo);
    at2(S::B2_OFF)[canon_offset(n, k, 16) / 2] = k == 0 ? hi : (k == 1 ? lo : __float2bfloat16_rn(0.0f));
  }
  for (int i = tid; i < kTileRows * 16; i += nth) {
    const int r = i / 16, k = i - r * 16;
    at2(S::ONES_OFF)[canon_offset(r, k, 16) / 2] = __float2bfloat16_rn(k < 2 ? 1.0f : 0.0f);
  }
  float *cv = reinterpret_cast<float *>(l2 + S::CV_OFF);
  for (int i = tid; i <= kCH; i += nth)
    cv[i] = i < kCH ? __bfloat162float(__float2bfloat16_rn(params[L.Cv + i])) : params[L.cv];
}

// ---- layer 1 -----------------------------------------------------------------------------------
// Warp-specialised, fed by the tensor-map copy engine.  An item is one K step (16 columns) of one
// 128-row tile.  One thread issues a tiled copy per item: 128 rows x 64 bytes of fp32 observations
// into a ring of shared-memory stages (64-byte swizzle, so that a thread reading its own row does
// not collide with its neighbours), never touching L1 or registers on the way.  Two converter
// groups of 128 threads (thread r = tile row r) alternate items: fp32 -> bf16 into a ring of
// operand buffers in the MMA's canonical K-major layout.  One thread issues the MMAs as the
// operand buffers fill and frees them by tcgen05.commit; four epilogue warps drain the two
// alternating accumulators.  Only mbarriers connect the roles, every wait is bounded.
// Rows are tiled per array (the T*E rows of `obs`, then the E rows of the last observation), so a
// tile never straddles the two; rows past an array's end come in as zeros and are never stored.
constexpr int kL1F32Stages = 5, kL1Bf16Stages = 3;
constexpr int kL1ConvGroups = 2, kL1ConvThreads = kL1ConvGroups * 128;
constexpr int kL1Threads = kL1ConvThreads + 128 + 64;  // converters, epilogue warps, copy warp, MMA warp
constexpr uint32_t kL1F32StageBytes = kTileRows * 16 * 4, kL1Bf16StageBytes = kTileRows * 16 * 2;

template <int N>
struct CriticL1Smem {
  using S = CriticShape<N>;
  alignas(1024) unsigned char c1[S::C1_BYTES];
  alignas(1024) unsigned char xf[kL1F32Stages][kL1F32StageBytes];
  alignas(128) unsigned char xb[kL1Bf16Stages][kL1Bf16StageBytes];
  alignas(8) uint64_t load_bar;
  alignas(8) uint64_t xf_full[kL1F32Stages], xf_empty[kL1F32Stages], xb_full[kL1Bf16Stages], xb_empty[kL1Bf16Stages];
  alignas(8) uint64_t acc_full[2], acc_empty[2];
  uint32_t tmem_base;
};
static_assert(CriticShape<4>::C1_BYTES % 1024 == 0, "the fp32 stages follow C1 on a swizzle-pattern boundary");

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Tiled 2-D copy global -> shared through a tensor map; x (innermost, in elements) must be a multiple of 4 floats.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
               "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
               : "memory");
}
__device__ __forceinline__ float4 lds_f32x4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}

template <int N>
__global__ void __launch_bounds__(kL1Threads, 1)
critic_l1_kernel(const __grid_constant__ CUtensorMap map_main, const __grid_constant__ CUtensorMap map_last, int tiles_main,
                 const unsigned char *__restrict__ image, unsigned char *__restrict__ h1, int n_tiles, int *status) {
  using S = CriticShape<N>;
  constexpr int KJ = S::KJ, K1 = S::K1, KS = K1 / 16;  // K steps per tile
  static_assert(KJ / 16 == KS - 1 && KJ % 16 == 4, "the ones columns open the second float4 of the last K step");
  extern __shared__ unsigned char smem_raw[];
  // the swizzle pattern of the fp32 stages repeats every 512 bytes of shared address: align by hand
  CriticL1Smem<N> &sm = *reinterpret_cast<CriticL1Smem<N> *>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u));
  const int tid = threadIdx.x, warp = tid / 32;
  if (tid == 0) {
    mbar_init(smem_u32(&sm.load_bar), 1);
    for (int i = 0; i < kL1F32Stages; ++i) {
      mbar_init(smem_u32(&sm.xf_full[i]), 1);
      mbar_init(smem_u32(&sm.xf_empty[i]), 4);  // one arrival per warp of the converting group
    }
    for (int i = 0; i < kL1Bf16Stages; ++i) {
      mbar_init(smem_u32(&sm.xb_full[i]), 4);
      mbar_init(smem_u32(&sm.xb_empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&sm.acc_full[i]), 1);
      mbar_init(smem_u32(&sm.acc_empty[i]), 4);  // one arrival per epilogue warp
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (tid == 0) {
    const uint32_t bar = smem_u32(&sm.load_bar);
    mbar_expect_tx(bar, S::C1_BYTES);
    constexpr uint32_t kChunk = 16384;
    for (uint32_t off = 0; off < S::C1_BYTES; off += kChunk)
      bulk_load(smem_u32(sm.c1 + off), image + off, S::C1_BYTES - off < kChunk ? S::C1_BYTES - off : kChunk, bar);
  }
  bool timed_out = !mbar_wait(smem_u32(&sm.load_bar), 0);
  timed_out = __syncthreads_or(timed_out) != 0;

  const uint32_t tmem_base = sm.tmem_base;
  const uint32_t xf_full0 = smem_u32(&sm.xf_full[0]), xf_empty0 = smem_u32(&sm.xf_empty[0]);
  const uint32_t xb_full0 = smem_u32(&sm.xb_full[0]), xb_empty0 = smem_u32(&sm.xb_empty[0]);
  const uint32_t acc_full0 = smem_u32(&sm.acc_full[0]), acc_empty0 = smem_u32(&sm.acc_empty[0]);
  const uint32_t xf0 = smem_u32(sm.xf[0]), xb0 = smem_u32(sm.xb[0]);
  // tiles of this CTA: blockIdx.x, blockIdx.x + gridDim.x, ...
  const int my_tiles = (n_tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
  const int n_items = my_tiles * KS;  // (tile, K step) pairs in order; item n uses fp32 stage n % 5, operand buffer n % 3

  if (timed_out) {
    // nothing was started
  } else if (tid < kL1ConvThreads) {
    // ---- converters: thread r of a group turns row r of an item into bf16 ---------------------
    const int g = tid / 128, r = tid % 128;
    const uint32_t src_row = static_cast<uint32_t>(r) * 64u, sw = static_cast<uint32_t>((r >> 1) & 3);  // 64-byte swizzle
    const uint32_t dst_row = static_cast<uint32_t>((r >> 3) * 256 + (r & 7) * 16);
#pragma unroll 1
    for (int n = g; n < n_items && !timed_out; n += kL1ConvGroups) {
      const int s = n % kL1F32Stages, b = n % kL1Bf16Stages;
      const bool last_step = n % KS == KS - 1;
      timed_out |= !mbar_wait(xf_full0 + 8u * s, (n / kL1F32Stages) & 1);
      const uint32_t src = xf0 + static_cast<uint32_t>(s) * kL1F32StageBytes + src_row;
      const float4 f0 = lds_f32x4(src + ((0u ^ sw) << 4));
      float4 f1 = lds_f32x4(src + ((1u ^ sw) << 4));
      const float4 f2 = lds_f32x4(src + ((2u ^ sw) << 4));
      const float4 f3 = lds_f32x4(src + ((3u ^ sw) << 4));
      if (last_step) f1 = make_float4(1.f, 1.f, 0.f, 0.f);  // the two ones columns that pick up c1 (the copy filled zeros)
      timed_out |= !mbar_wait(xb_empty0 + 8u * b, ((n / kL1Bf16Stages) & 1) ^ 1);  // the MMA that read this buffer is done
      timed_out = __any_sync(0xFFFFFFFFu, timed_out);  // the warp leaves together
      if (timed_out) break;
      const uint32_t dst = xb0 + static_cast<uint32_t>(b) * kL1Bf16StageBytes + dst_row;
      sts_v4(dst, pack_bf16(f0.x, f0.y), pack_bf16(f0.z, f0.w), pack_bf16(f1.x, f1.y), pack_bf16(f1.z, f1.w));
      sts_v4(dst + 128, pack_bf16(f2.x, f2.y), pack_bf16(f2.z, f2.w), pack_bf16(f3.x, f3.y), pack_bf16(f3.z, f3.w));
      fence_async_smem();
      __syncwarp();
      if ((tid & 31) == 0) {
        mbar_arrive(xb_full0 + 8u * b);
        mbar_arrive(xf_empty0 + 8u * s);  // after the stores, which needed the loaded values: the stage has been read
      }
    }
  } else if (tid < kL1ConvThreads + 128) {
    // ---- epilogue warps: ReLU, bf16, the row goes out in the operand layout of layer 2 -----------
    const int row = tid - kL1ConvThreads;  // 0..127: tile row and tensor-memory lane
    const uint32_t lane_off = static_cast<uint32_t>((row / 32) * 32) << 16;
    for (int kt = 0; kt < my_tiles && !timed_out; ++kt) {
      const int a = kt & 1;
      const long long tile = static_cast<long long>(blockIdx.x) + static_cast<long long>(kt) * gridDim.x;
      timed_out |= !mbar_wait(acc_full0 + 8u * a, (kt >> 1) & 1);
      tc_fence_after();
      const uint32_t acc = tmem_base + static_cast<uint32_t>(a * kCH);
      unsigned char *tile_out = h1 + static_cast<size_t>(tile) * S::H1_TILE_BYTES;
      uint32_t ra[32], pk[16];
#pragma unroll 1
      for (int c0 = 0; c0 < kCH; c0 += 32) {
        tmem_ld32_nowait(acc + lane_off + static_cast<uint32_t>(c0), ra);
        tmem_ld_wait();
        relu_pack32(ra, pk);
#pragma unroll
        for (int q = 0; q < 4; ++q)
          *reinterpret_cast<uint4 *>(tile_out + canon_offset(row, c0 + 8 * q, kCH)) =
              make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
      }
      tc_fence_before();
      __syncwarp();
      if ((tid & 31) == 0) mbar_arrive(acc_empty0 + 8u * a);
    }
  } else if (tid == kL1ConvThreads + 128) {
    // ---- the copy thread ----------------------------------------------------------------------
    int n = 0;
    for (int kt = 0; kt < my_tiles && !timed_out; ++kt) {
      const int tile = static_cast<int>(blockIdx.x) + kt * static_cast<int>(gridDim.x);
      const bool in_main = tile < tiles_main;
      const CUtensorMap *map = in_main ? &map_main : &map_last;
      const int y = (in_main ? tile : tile - tiles_main) * kTileRows;
      for (int ks = 0; ks < KS && !timed_out; ++ks, ++n) {
        const int s = n % kL1F32Stages;
        timed_out |= !mbar_wait(xf_empty0 + 8u * s, ((n / kL1F32Stages) & 1) ^ 1);
        if (timed_out) break;
        mbar_expect_tx(xf_full0 + 8u * s, kL1F32StageBytes);
        tma_load_2d(xf0 + static_cast<uint32_t>(s) * kL1F32StageBytes, map, ks * 16, y, xf_full0 + 8u * s);
      }
    }
    if (timed_out)  // let the copies still in flight land before the block goes away
      for (int j = n > kL1F32Stages ? n - kL1F32Stages : 0; j < n; ++j)
        mbar_wait(xf_full0 + 8u * (j % kL1F32Stages), (j / kL1F32Stages) & 1);
  } else if (tid == kL1ConvThreads + 128 + 32) {
    // ---- the MMA-issuing thread -----------------------------------------------------------------
    const uint32_t c1_addr = smem_u32(sm.c1);
    int n = 0;
    for (int kt = 0; kt < my_tiles && !timed_out; ++kt) {
      const int a = kt & 1;
      timed_out |= !mbar_wait(acc_empty0 + 8u * a, ((kt >> 1) & 1) ^ 1);  // the epilogue has drained this accumulator
      tc_fence_after();
      const uint32_t acc = tmem_base + static_cast<uint32_t>(a * kCH);
      for (int ks = 0; ks < KS && !timed_out; ++ks, ++n) {
        const int b = n % kL1Bf16Stages;
        timed_out |= !mbar_wait(xb_full0 + 8u * b, (n / kL1Bf16Stages) & 1);
        if (timed_out) break;
        tc_fence_after();
        mma_bf16(acc, smem_desc(xb0 + static_cast<uint32_t>(b) * kL1Bf16StageBytes, 128, 256),
                 smem_desc(c1_addr + static_cast<uint32_t>(ks) * 256, 128, K1 * 16), instr_desc(kTileRows, kCH), ks > 0 ? 1u : 0u);
        mma_commit(xb_empty0 + 8u * b);  // frees the buffer when this MMA has read it
      }
      if (!timed_out) mma_commit(acc_full0 + 8u * a);
    }
  }
  if (timed_out) atomicExch(status, kStatusTimeout);
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

// ---- layer 2 and the value head ----------------------------------------------------------------
template <int N>
struct CriticL2Smem {
  using S = CriticShape<N>;
  alignas(128) unsigned char w[S::L2_BYTES];
  alignas(128) unsigned char a[S::H1_TILE_BYTES];
  alignas(8) uint64_t w_bar;
  alignas(8) uint64_t load_bar[2];  // round k's tile completes load_bar[k % 2]: each group has its own
  alignas(8) uint64_t mma_bar[2];
  uint32_t tmem_base;
};

template <int N>
__global__ void __launch_bounds__(2 * kGroupThreads, 1)
critic_l2_kernel(const unsigned char *__restrict__ h1, const unsigned char *__restrict__ image, float *__restrict__ values,
                 long long rows_main, long long rows_total, int tiles_main, int n_tiles, int *status) {
  using S = CriticShape<N>;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  CriticL2Smem<N> &sm = *reinterpret_cast<CriticL2Smem<N> *>(smem_raw);
  const int tid = threadIdx.x, g = tid / kGroupThreads, row = tid % kGroupThreads, warp = tid / 32;
  const uint32_t load_bar0 = smem_u32(&sm.load_bar[0]);
  auto load_tile = [&](int tile, int round) {  // one thread: the tile's 64 KB in four bulk copies
    const uint32_t lb = load_bar0 + 8u * (round & 1);
    mbar_expect_tx(lb, S::H1_TILE_BYTES);
    for (uint32_t off = 0; off < S::H1_TILE_BYTES; off += 16384)
      bulk_load(smem_u32(sm.a + off), h1 + static_cast<size_t>(tile) * S::H1_TILE_BYTES + off, 16384, lb);
  };
  if (tid == 0) {
    mbar_init(smem_u32(&sm.w_bar), 1);
    mbar_init(load_bar0, 1);
    mbar_init(load_bar0 + 8, 1);
    mbar_init(smem_u32(&sm.mma_bar[0]), 1);
    mbar_init(smem_u32(&sm.mma_bar[1]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (tid == 0) {
    const uint32_t bar = smem_u32(&sm.w_bar);
    mbar_expect_tx(bar, S::L2_BYTES);
    for (uint32_t off = 0; off < S::L2_BYTES; off += 16384)
      bulk_load(smem_u32(sm.w + off), image + off, S::L2_BYTES - off < 16384 ? S::L2_BYTES - off : 16384, bar);
    if (static_cast<int>(blockIdx.x) < n_tiles) load_tile(blockIdx.x, 0);  // round 0 belongs to group 0
  }
  bool timed_out = !mbar_wait(smem_u32(&sm.w_bar), 0);
  timed_out = __syncthreads_or(timed_out) != 0;

  const uint32_t tmem_base = sm.tmem_base;
  const uint32_t acc = tmem_base + static_cast<uint32_t>(g * kCH);
  const uint32_t lane_off = static_cast<uint32_t>((row / 32) * 32) << 16;
  const uint32_t w_addr = smem_u32(sm.w), a_addr = smem_u32(sm.a), cv_addr = w_addr + S::CV_OFF;
  const uint32_t mma_bar = smem_u32(&sm.mma_bar[g]);

  // round k of this CTA works on tile blockIdx.x + k * gridDim.x and belongs to group k % 2
  for (int k = g; !timed_out; k += 2) {
    const int tile = blockIdx.x + k * static_cast<int>(gridDim.x);
    if (tile >= n_tiles) break;
    timed_out |= !mbar_wait(load_bar0 + 8u * g, (k >> 1) & 1);  // this round's tile has landed
    if (row == 0 && !timed_out) {
      tc_fence_after();
      constexpr uint32_t idesc = instr_desc(kTileRows, kCH);
      mma_bf16(acc, smem_desc(w_addr + S::ONES_OFF, 128, 256), smem_desc(w_addr + S::B2_OFF, 128, 256), idesc, 0);
#pragma unroll
      for (int j = 0; j < kCH / 16; ++j)
        mma_bf16(acc, smem_desc(a_addr + j * 256, 128, kCH * 16), smem_desc(w_addr + S::C2_OFF + j * 256, 128, kCH * 16),
                 idesc, 1);
      mma_commit(mma_bar);
    }
    if (!timed_out) timed_out |= !mbar_wait(mma_bar, (k >> 1) & 1);
    // the tile buffer is free: fetch the next round's tile (the other group's) behind this epilogue
    if (row == 0 && !timed_out && tile + static_cast<int>(gridDim.x) < n_tiles) load_tile(tile + gridDim.x, k + 1);
    tc_fence_after();
    float v = 0.0f;
    uint32_t ra[32];
#pragma unroll 1
    for (int c0 = 0; c0 < kCH; c0 += 32) {
      tmem_ld32_nowait(acc + lane_off + static_cast<uint32_t>(c0), ra);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const uint32_t p = relu_pack_bf16(ra[2 * i], ra[2 * i + 1]);  // h2 rounded to bf16, as the operands of the head are
        v = fmaf(__uint_as_float(p << 16), lds_f32(cv_addr + 4u * (c0 + 2 * i)), v);
        v = fmaf(__uint_as_float(p & 0xFFFF0000u), lds_f32(cv_addr + 4u * (c0 + 2 * i + 1)), v);
      }
    }
    v += lds_f32(cv_addr + 4u * kCH);
    // layer 1 tiles the two observation arrays separately: main tiles first, then those of the last observation
    const bool in_main = tile < tiles_main;
    const long long r_loc = static_cast<long long>(in_main ? tile : tile - tiles_main) * kTileRows + row;
    const long long r_idx = in_main ? r_loc : rows_main + r_loc;
    if (r_loc < (in_main ? rows_main : rows_total - rows_main) && !timed_out) {
      float *out = values + r_idx * N;
#pragma unroll
      for (int n = 0; n < N; ++n) out[n] = v;
    }
    tc_fence_before();
    if (group_any(g, timed_out)) timed_out = true;
  }
  if (timed_out && row == 0) atomicExch(status, kStatusTimeout);
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

// Tensor map of a row-major fp32 matrix [rows][width] for boxes of 128 rows x 16 columns (64 bytes, 64-byte swizzle);
// elements outside the matrix read as zero.  The encoder is a driver entry point fetched through the runtime.
bool encode_obs_map(CUtensorMap *map, const float *base, long long rows, int width) {
  using Fn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                          const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                          CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static Fn encode = [] {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<Fn>(p);
  }();
  if (!encode || rows < 1 || reinterpret_cast<uintptr_t>(base) % 16 != 0 || (width * sizeof(float)) % 16 != 0) return false;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(width), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(width) * sizeof(float)};
  const cuuint32_t box[2] = {16, kTileRows}, elem[2] = {1, 1};
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(base), dims, strides, box, elem,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

size_t critic_weight_bytes(const mava_config_t &cfg) {
  return find_variant(cfg) == 3 ? CriticShape<4>::IMAGE_BYTES : 16;
}

size_t critic_hidden_bytes(const mava_config_t &cfg) {
  if (find_variant(cfg) != 3) return 16;
  const long long rows = static_cast<long long>(cfg.max_T) * cfg.n_envs;
  const long long tiles = (rows + kTileRows - 1) / kTileRows + (cfg.n_envs + kTileRows - 1) / kTileRows;
  return static_cast<size_t>(tiles) * CriticShape<4>::H1_TILE_BYTES;
}

cudaError_t launch_critic_tc(mava_rollout *h, const float *params_dev, int32_t T) {
  if (h->variant != 3 || !h->d_critic || !h->d_critic_h1 || !h->d_obs_last) return cudaErrorNotSupported;
  using S = CriticShape<4>;
  unsigned char *image = static_cast<unsigned char *>(h->d_critic);
  prep_critic_kernel<4><<<128, 256, 0, h->stream>>>(params_dev, image, param_layout(h->cfg, h->D, 1));
  h->launches += 1;
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  int sms = 0;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->device);
  if (err != cudaSuccess) return err;
  const long long rows_main = static_cast<long long>(T) * h->cfg.n_envs, rows_total = rows_main + h->cfg.n_envs;
  const int tiles_main = static_cast<int>((rows_main + kTileRows - 1) / kTileRows);
  const int n_tiles = tiles_main + (h->cfg.n_envs + kTileRows - 1) / kTileRows;
  {
    CUtensorMap map_main, map_last;
    if (!encode_obs_map(&map_main, h->buf.obs, rows_main, S::KJ) || !encode_obs_map(&map_last, h->d_obs_last, h->cfg.n_envs, S::KJ))
      return cudaErrorInvalidValue;
    auto kern = critic_l1_kernel<4>;
    const size_t smem = sizeof(CriticL1Smem<4>) + 1024;  // room to align the struct by hand
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (err != cudaSuccess) return err;
    const int ctas = n_tiles < sms ? n_tiles : sms;
    kern<<<ctas, kL1Threads, smem, h->stream>>>(map_main, map_last, tiles_main, image, static_cast<unsigned char *>(h->d_critic_h1),
                                                n_tiles, h->d_status);
    h->launches += 1;
    err = cudaGetLastError();
    if (err != cudaSuccess) return err;
  }
  {
    auto kern = critic_l2_kernel<4>;
    const size_t smem = sizeof(CriticL2Smem<4>);
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (err != cudaSuccess) return err;
    const int ctas = n_tiles < sms ? n_tiles : sms;
    kern<<<ctas, 2 * kGroupThreads, smem, h->stream>>>(static_cast<const unsigned char *>(h->d_critic_h1), image + S::C1_BYTES,
                                                       h->buf.values, rows_main, rows_total, tiles_main, n_tiles, h->d_status);
    h->launches += 1;
    err = cudaGetLastError();
  }
  return err;
}

}  // namespace mava
