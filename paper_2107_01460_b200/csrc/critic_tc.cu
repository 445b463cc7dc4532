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
// Warp-specialised.  Four producer groups of three warps each own one stage of a ring of bf16 A
// buffers: group g loads item g, g + 4, ... (an item is one 48-column chunk of one 128-row tile)
// into registers, converts it into its stage and at once starts the loads of its next item, so four
// items of loads are in flight per SM with a single item per thread.  One thread issues the MMAs as
// the stages fill and frees them by tcgen05.commit; four epilogue warps drain the two alternating
// accumulators.  Only mbarriers connect the roles, every wait is bounded.
constexpr int kL1Stages = 4, kL1GroupThreads = 96, kL1Producers = kL1Stages * kL1GroupThreads;
constexpr int kL1Threads = kL1Producers + 128 + 32;  // producers, epilogue warps, the issuing warp

template <int N>
struct CriticL1Smem {
  using S = CriticShape<N>;
  alignas(128) unsigned char c1[S::C1_BYTES];
  alignas(128) unsigned char abuf[kL1Stages][S::A_BUF_BYTES];
  alignas(8) uint64_t load_bar;
  alignas(8) uint64_t full[kL1Stages], empty[kL1Stages], acc_full[2], acc_empty[2];
  uint32_t tmem_base;
};

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

template <int N>
__global__ void __launch_bounds__(kL1Threads, 1)
critic_l1_kernel(const float *__restrict__ obs, const float *__restrict__ obs_last, long long rows_main,
                 long long rows_total, const unsigned char *__restrict__ image, unsigned char *__restrict__ h1, int n_tiles,
                 int *status) {
  using S = CriticShape<N>;
  constexpr int KJ = S::KJ, K1 = S::K1, CHUNK = S::CHUNK, NCHUNK = S::NCHUNK;
  constexpr int V = CHUNK / 4;        // float4 per row and chunk
  constexpr int Q = kTileRows / 8;    // float4 per producer thread and item: rows r0, r0 + 8, ...
  static_assert(V * 8 == kL1GroupThreads, "a group covers eight rows of a chunk per pass");
  extern __shared__ __align__(128) unsigned char smem_raw[];
  CriticL1Smem<N> &sm = *reinterpret_cast<CriticL1Smem<N> *>(smem_raw);
  const int tid = threadIdx.x, warp = tid / 32;
  if (tid == 0) {
    mbar_init(smem_u32(&sm.load_bar), 1);
    for (int i = 0; i < kL1Stages; ++i) {
      mbar_init(smem_u32(&sm.full[i]), kL1GroupThreads / 32);  // one arrival per warp of the stage's group
      mbar_init(smem_u32(&sm.empty[i]), 1);
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
  const uint32_t full0 = smem_u32(&sm.full[0]), empty0 = smem_u32(&sm.empty[0]);
  const uint32_t acc_full0 = smem_u32(&sm.acc_full[0]), acc_empty0 = smem_u32(&sm.acc_empty[0]);
  const uint32_t abuf0 = smem_u32(sm.abuf[0]);
  // tiles of this CTA: blockIdx.x, blockIdx.x + gridDim.x, ...
  const int my_tiles = (n_tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
  const int n_items = my_tiles * NCHUNK;  // (tile, chunk) pairs in order; item n uses ring stage n % kL1Stages

  if (!timed_out && tid < kL1Producers) {
    // ---- producers --------------------------------------------------------------------------
    // Thread t of a group takes float4 v = t % 12 of rows r0 + 8 q (r0 = t / 12): consecutive threads
    // read consecutive 16 bytes of a row, and every address is a per-thread base plus a constant.
    const int g = tid / kL1GroupThreads, t = tid - g * kL1GroupThreads;
    const int v = t % V, r0 = t / V;
    const uint32_t goff = static_cast<uint32_t>(r0 * KJ + 4 * v);  // in floats, within the tile's block of rows
    const uint32_t sdst = abuf0 + static_cast<uint32_t>(g) * S::A_BUF_BYTES +
                          static_cast<uint32_t>(((4 * v) >> 3) * S::A_LBO + r0 * 16 + ((4 * v) & 7) * 2);
    // in the last chunk: the two ones columns that pick up c1, and the zero columns after them
    const bool ones = (NCHUNK - 1) * CHUNK + 4 * v == KJ, past = (NCHUNK - 1) * CHUNK + 4 * v > KJ;
    const uint32_t full_bar = full0 + 8u * g, empty_bar = empty0 + 8u * g;
    int n = g, kt = 0, c = g;  // this group's next item and its (tile, chunk)
    static_assert(kL1Stages <= S::NCHUNK, "the first items of all groups lie in the first tile");
    float4 d[Q];
    auto load_item = [&]() {
      const long long row0 = (static_cast<long long>(blockIdx.x) + static_cast<long long>(kt) * gridDim.x) * kTileRows;
      const bool in_main = row0 + kTileRows <= rows_main;
      const bool in_last = row0 >= rows_main && row0 + kTileRows <= rows_total;
      const bool last_chunk = c == NCHUNK - 1;
      if (last_chunk && (ones || past)) {
#pragma unroll
        for (int q = 0; q < Q; ++q) d[q] = make_float4(ones ? 1.f : 0.f, ones ? 1.f : 0.f, 0.f, 0.f);
      } else if (in_main || in_last) {
        // the tile lies wholly inside one of the two observation arrays: a contiguous block of rows
        const float *src = (in_main ? obs + row0 * KJ : obs_last + (row0 - rows_main) * KJ) + c * CHUNK + goff;
#pragma unroll
        for (int q = 0; q < Q; ++q) d[q] = __ldg(reinterpret_cast<const float4 *>(src + q * 8 * KJ));
      } else {
#pragma unroll
        for (int q = 0; q < Q; ++q) {
          const long long r_idx = row0 + r0 + 8 * q;
          d[q] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (r_idx < rows_total)
            d[q] = __ldg(reinterpret_cast<const float4 *>(
                (r_idx < rows_main ? obs + r_idx * KJ : obs_last + (r_idx - rows_main) * KJ) + c * CHUNK + 4 * v));
        }
      }
    };
    if (n < n_items) load_item();
#pragma unroll 1
    for (uint32_t it = 0; n < n_items && !timed_out; ++it) {
      timed_out |= !mbar_wait(empty_bar, (it & 1) ^ 1);  // the MMAs that read this stage are done
#pragma unroll
      for (int q = 0; q < Q; ++q)
        asm volatile("st.shared.v2.u32 [%0], {%1, %2};" ::"r"(sdst + q * S::A_SBO), "r"(pack_bf16(d[q].x, d[q].y)),
                     "r"(pack_bf16(d[q].z, d[q].w))
                     : "memory");
      fence_async_smem();
      __syncwarp();
      if ((tid & 31) == 0) mbar_arrive(full_bar);
      n += kL1Stages;
      c += kL1Stages;
      if (c >= NCHUNK) { c -= NCHUNK; ++kt; }
      if (n < n_items) load_item();
    }
  } else if (!timed_out && tid >= kL1Producers + 128) {
    // ---- the issuing thread -----------------------------------------------------------------
    if (tid == kL1Producers + 128) {
      const uint32_t c1_addr = smem_u32(sm.c1);
      for (int kt = 0; kt < my_tiles && !timed_out; ++kt) {
        const int a = kt & 1;
        timed_out |= !mbar_wait(acc_empty0 + 8u * a, ((kt >> 1) & 1) ^ 1);  // the epilogue has drained this accumulator
        tc_fence_after();
        const uint32_t acc = tmem_base + static_cast<uint32_t>(a * kCH);
        for (int c = 0; c < NCHUNK && !timed_out; ++c) {
          const int n = kt * NCHUNK + c, s2 = n % kL1Stages;
          timed_out |= !mbar_wait(full0 + 8u * s2, (n / kL1Stages) & 1);
          tc_fence_after();
          const uint32_t abuf = abuf0 + static_cast<uint32_t>(s2) * S::A_BUF_BYTES;
#pragma unroll
          for (int j = 0; j < CHUNK / 16; ++j)
            mma_bf16(acc, smem_desc(abuf + j * 2 * S::A_LBO, S::A_LBO, S::A_SBO),
                     smem_desc(c1_addr + (c * (CHUNK / 16) + j) * 256, 128, K1 * 16), instr_desc(kTileRows, kCH),
                     (c > 0 || j > 0) ? 1u : 0u);
          mma_commit(empty0 + 8u * s2);  // frees the stage when these MMAs have read it
        }
        mma_commit(acc_full0 + 8u * a);
      }
    }
  } else if (!timed_out) {
    // ---- epilogue warps: ReLU, bf16, the row goes out in the operand layout of layer 2 -----------
    const int row = tid - kL1Producers;  // 0..127: tile row and tensor-memory lane
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
                 long long rows_total, int n_tiles, int *status) {
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
    const long long r_idx = static_cast<long long>(tile) * kTileRows + row;
    if (r_idx < rows_total && !timed_out) {
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

}  // namespace

size_t critic_weight_bytes(const mava_config_t &cfg) {
  return find_variant(cfg) == 3 ? CriticShape<4>::IMAGE_BYTES : 16;
}

size_t critic_hidden_bytes(const mava_config_t &cfg) {
  if (find_variant(cfg) != 3) return 16;
  const long long rows = static_cast<long long>(cfg.max_T + 1) * cfg.n_envs;
  return static_cast<size_t>((rows + kTileRows - 1) / kTileRows) * CriticShape<4>::H1_TILE_BYTES;
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
  const int n_tiles = static_cast<int>((rows_total + kTileRows - 1) / kTileRows);
  {
    auto kern = critic_l1_kernel<4>;
    const size_t smem = sizeof(CriticL1Smem<4>);
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (err != cudaSuccess) return err;
    const int ctas = n_tiles < sms ? n_tiles : sms;
    kern<<<ctas, kL1Threads, smem, h->stream>>>(h->buf.obs, h->d_obs_last, rows_main, rows_total, image,
                                                static_cast<unsigned char *>(h->d_critic_h1), n_tiles, h->d_status);
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
                                                       h->buf.values, rows_total, n_tiles, h->d_status);
    h->launches += 1;
    err = cudaGetLastError();
  }
  return err;
}

}  // namespace mava
