// Centralised critic (MAPPO) on the tensor cores, as one batched kernel over the stored
// trajectory: the critic's value does not feed the next environment step, so it is taken off the
// rollout's serial chain and computed for all (T+1)*E environment-steps at once:
//   h1 = relu(X C1^T + c1), X = the N observations of an environment-step concatenated (N*D fp32,
//        contiguous in the time-major obs array), brought in by tensor-map copies and rounded to bf16;
//   v  = Cv relu(h1 C2^T + c2) + cv, h1 and h2 rounded to bf16 as the operands of the next layer are.
// Pairs of SMs share the two weight matrices (tcgen05 cta_group::2), h1 stays in tensor memory.
// Every mbarrier wait is bounded; a role that gives up records kStatusTimeout and leaves.
#include "common.cuh"
#include "layout.h"
#include "tc_common.cuh"
#include "tmap.cuh"

namespace mava {
namespace {

constexpr int kCH = 256;  // hidden width of the compiled critic


template <int N>
struct CriticShape {
  static constexpr int D = kObsFixed + N;
  static constexpr int KJ = N * D;                        // joint observation width
  static constexpr int K1 = (KJ + 2 + 15) / 16 * 16;      // + two ones columns that carry c1
  static_assert(KJ % 4 == 0, "rows are whole 16-byte pieces");
  static constexpr uint32_t C1_BYTES = kCH * K1 * 2;
  // after C1: C2 | Cv (bf16-rounded, as fp32), cv, three unused floats, c2 (fp32)
  static constexpr uint32_t C2_OFF = 0, C2_BYTES = kCH * kCH * 2;
  static constexpr uint32_t CV_OFF = C2_OFF + C2_BYTES, CV_BYTES = (2 * kCH + 4) * 4;
  static constexpr uint32_t L2_BYTES = CV_OFF + CV_BYTES;
  static constexpr uint32_t IMAGE_BYTES = C1_BYTES + L2_BYTES;
};

// fp32 parameters -> the operand images: C1 and C2 as bf16 in the canonical K-major layout (output
// units 0..127 in the first half of each image, 128..255 in the second), c1 split into bf16 hi + lo
// in two spare K columns of C1, and the fp32 vectors the epilogue of layer 2 needs.
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
  for (int i = tid; i < kCH * kCH; i += nth) {
    const int n = i / kCH, k = i - n * kCH;
    reinterpret_cast<__nv_bfloat16 *>(l2 + S::C2_OFF)[canon_offset(n, k, kCH) / 2] =
        __float2bfloat16_rn(params[L.C2 + static_cast<size_t>(n) * kCH + k]);
  }
  float *cv = reinterpret_cast<float *>(l2 + S::CV_OFF);
  for (int i = tid; i < 2 * kCH + 4; i += nth)
    cv[i] = i < kCH ? __bfloat162float(__float2bfloat16_rn(params[L.Cv + i]))
                    : (i == kCH ? params[L.cv] : (i < kCH + 4 ? 0.0f : params[L.c2 + i - kCH - 4]));
}

// ---- both layers in one kernel, on pairs of SMs --------------------------------------------------
// A cluster of two CTAs (two SMs) works on 256 consecutive environment-steps, 128 per CTA, with
// tcgen05.mma.cta_group::2: M = 256 (each CTA's rows accumulate in its own tensor memory), and each
// CTA holds half of the output units of C1 and C2 in shared memory (86 + 64 KB), so both layers'
// weights are resident and the hidden activations never leave the chip:
//   copy thread    tiled tensor-map copies, one K step (128 rows x 16 fp32 columns, 64-byte swizzle)
//                  at a time, into a ring of shared-memory stages;
//   converters     two groups of 128 threads (thread r = row r) alternate K steps: fp32 -> bf16 into
//                  a ring of operand buffers (canonical K-major layout); they report to the leader;
//   MMA thread     of the leader CTA (cluster rank 0) only: layer 1 (N = 256) as the buffers of BOTH
//                  CTAs fill; then, once both CTAs' epilogue warps have put relu(h1) as bf16 back into
//                  tensor memory, layer 2 with h1 as the A operand straight from tensor memory, in two
//                  passes of N = 128 into a separate accumulator, the second pass slipped in between
//                  the next tile's layer-1 steps as soon as the first has been drained;
//   epilogue warps eight per CTA (a lane quarter and a column half each): layer 1 into h1, then the two
//                  passes of layer 2 into the value (bias, ReLU, bf16 rounding, dot with Cv), written
//                  to the N slots of the environment-step.
// Barriers the leader waits on collect arrivals from both CTAs (remote mbarrier arrive); barriers the
// other roles wait on are signalled in both CTAs by one multicast tcgen05.commit.  Every mbarrier
// wait is bounded; whoever gives up records kStatusTimeout and walks to the common exit.
// Rows are tiled per array (the T*E rows of `obs`, then the E rows of the last observation), so a
// tile never straddles the two; rows past an array's end come in as zeros and are never stored.
constexpr int kConvGroups = 2, kConvThreads = kConvGroups * 128, kEpiThreads = 256;
constexpr int kCriticThreads = kConvThreads + kEpiThreads + 64;  // converters, epilogue warps, copy warp, MMA warp
constexpr uint32_t kXfBytes = kTileRows * 16 * 4, kXbBytes = kTileRows * 16 * 2;
// tensor-memory columns: layer-1 accumulator 0..255, h1 (two bf16 per column) 256..383, layer-2 accumulator 384..511
constexpr uint32_t kHidCol = kCH, kAcc2Col = kCH + kCH / 2;

template <int N, int XF, int XB, int G>
struct CriticSmem {
  using S = CriticShape<N>;
  alignas(1024) unsigned char c1[S::C1_BYTES / 2];
  alignas(1024) unsigned char xf[XF][kXfBytes];
  alignas(128) unsigned char c2[S::C2_BYTES / 2];
  alignas(128) unsigned char xb[XB][G * kXbBytes];  // an operand buffer holds G consecutive K steps
  alignas(16) unsigned char cv[S::CV_BYTES];
  float part[2][kTileRows];  // value partial sums of the upper column half, by tile parity
  alignas(8) uint64_t load_bar;
  alignas(8) uint64_t xf_full[XF], xf_empty[XF];
  alignas(8) uint64_t xb_full[XB];    // the leader's copy collects both CTAs' converters
  alignas(8) uint64_t xb_empty[XB];   // signalled in both CTAs by the leader's commit
  alignas(8) uint64_t acc1_full, acc2_full;  // signalled in both CTAs by the leader's commit
  alignas(8) uint64_t h1_full, acc2_free;    // the leader's copies collect both CTAs' epilogue warps
  alignas(8) uint64_t part_full[2];
  uint32_t tmem_base;
};
static_assert((CriticShape<4>::C1_BYTES / 2) % 1024 == 0, "the fp32 stages follow C1 on a swizzle-pattern boundary");

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ float4 lds_f32x4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address, in the cluster's shared window, of the same shared-memory offset in the CTA of rank `rank`.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// The pair's MMA: issued by one thread of the leader; the descriptors name the same shared-memory
// offsets in both CTAs, d_tmem (and a_tmem) the same tensor-memory columns.
__device__ __forceinline__ void mma2_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma2_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives, once the pair's MMAs issued so far are complete, on the barrier at this offset in both CTAs.
__device__ __forceinline__ void mma2_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
               "h"(static_cast<uint16_t>(3))
               : "memory");
}

template <int N, int XF, int XB, int G>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kCriticThreads, 1)
critic_kernel(const __grid_constant__ CUtensorMap map_main, const __grid_constant__ CUtensorMap map_last, int tiles_main,
              long long rows_main, long long rows_total, const unsigned char *__restrict__ image, float *__restrict__ values,
              int n_tiles, int *status) {
  using S = CriticShape<N>;
  constexpr int KJ = S::KJ, K1 = S::K1, KS = K1 / 16;  // K steps of layer 1 per tile
  static_assert(KJ / 16 == KS - 1 && KJ % 16 == 4, "the ones columns open the second float4 of the last K step");
  // The tensor-map copies of different stages complete in any order.  A parity wait on a stage's barrier is only
  // safe for the thread group that also consumed the stage's previous phase (a group that did not could arrive two
  // phases early and be let through), so a stage must always fall to the same converter group.
  static_assert(XF % (kConvGroups * G) == 0, "every fp32 stage belongs to one converter group");
  extern __shared__ unsigned char smem_raw[];
  // the swizzle pattern of the fp32 stages repeats every 512 bytes of shared address: align by hand
  // (the offset is the same in both CTAs, as the MMA's descriptors and the multicast commits need)
  CriticSmem<N, XF, XB, G> &sm =
      *reinterpret_cast<CriticSmem<N, XF, XB, G> *>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u));
  const int tid = threadIdx.x, warp = tid / 32;
  const uint32_t rank = cluster_ctarank();
  if (tid == 0) {
    mbar_init(smem_u32(&sm.load_bar), 1);
    for (int i = 0; i < XF; ++i) {
      mbar_init(smem_u32(&sm.xf_full[i]), 1);
      mbar_init(smem_u32(&sm.xf_empty[i]), 4);  // one arrival per warp of the converting group
    }
    for (int i = 0; i < XB; ++i) {
      mbar_init(smem_u32(&sm.xb_full[i]), 8);   // the converting group's warps of both CTAs
      mbar_init(smem_u32(&sm.xb_empty[i]), 1);
    }
    mbar_init(smem_u32(&sm.acc1_full), 1);
    mbar_init(smem_u32(&sm.acc2_full), 1);
    mbar_init(smem_u32(&sm.h1_full), 16);    // the epilogue warps of both CTAs
    mbar_init(smem_u32(&sm.acc2_free), 16);
    mbar_init(smem_u32(&sm.part_full[0]), 4);
    mbar_init(smem_u32(&sm.part_full[1]), 4);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers are initialised before anything arrives on them
  tc_fence_after();
  if (tid == 0) {
    // this CTA's half of the output units of C1 and C2; Cv, cv and c2
    const uint32_t bar = smem_u32(&sm.load_bar);
    const unsigned char *l2 = image + S::C1_BYTES;
    mbar_expect_tx(bar, S::C1_BYTES / 2 + S::C2_BYTES / 2 + S::CV_BYTES);
    auto load = [&](void *dst, const unsigned char *src, uint32_t bytes) {
      for (uint32_t off = 0; off < bytes; off += 16384)
        bulk_load(smem_u32(static_cast<unsigned char *>(dst) + off), src + off, bytes - off < 16384 ? bytes - off : 16384, bar);
    };
    load(sm.c1, image + rank * (S::C1_BYTES / 2), S::C1_BYTES / 2);
    load(sm.c2, l2 + S::C2_OFF + rank * (S::C2_BYTES / 2), S::C2_BYTES / 2);
    load(sm.cv, l2 + S::CV_OFF, S::CV_BYTES);
  }
  bool timed_out = !mbar_wait(smem_u32(&sm.load_bar), 0);
  timed_out = __syncthreads_or(timed_out) != 0;

  const uint32_t tmem_base = sm.tmem_base;
  const uint32_t xf_full0 = smem_u32(&sm.xf_full[0]), xf_empty0 = smem_u32(&sm.xf_empty[0]);
  const uint32_t xb_full0 = smem_u32(&sm.xb_full[0]), xb_empty0 = smem_u32(&sm.xb_empty[0]);
  const uint32_t acc1_full = smem_u32(&sm.acc1_full), acc2_full = smem_u32(&sm.acc2_full);
  const uint32_t xf0 = smem_u32(sm.xf[0]), xb0 = smem_u32(sm.xb[0]);
  // the leader's copies of the barriers that collect both CTAs
  const uint32_t lead_xb_full0 = map_to_cta(xb_full0, 0), lead_h1_full = map_to_cta(smem_u32(&sm.h1_full), 0),
                 lead_acc2_free = map_to_cta(smem_u32(&sm.acc2_free), 0);
  // pair-tiles (256 rows) of this cluster: pair, pair + n_pairs, ...; this CTA takes tile 2 * pair-tile + rank
  const int pair = static_cast<int>(blockIdx.x) / 2, n_pairs = static_cast<int>(gridDim.x) / 2;
  const int n_pair_tiles = (n_tiles + 1) / 2;
  const int my_tiles = pair < n_pair_tiles ? (n_pair_tiles - pair + n_pairs - 1) / n_pairs : 0;
  // K steps of all this CTA's tiles in order: step n uses fp32 stage n % XF; G consecutive steps (whatever
  // tiles they belong to) form item n / G, which uses operand buffer (n / G) % XB and is one hand-over
  const int n_steps = my_tiles * KS, n_items = (n_steps + G - 1) / G;
  auto tile_of = [&](int kt) { return 2 * (pair + kt * n_pairs) + static_cast<int>(rank); };

  if (timed_out) {
    // nothing was started
  } else if (tid < kConvThreads) {
    // ---- converters: thread r of a group turns row r of an item into bf16 ---------------------
    const int g = tid / 128, r = tid % 128;
    const uint32_t src_row = static_cast<uint32_t>(r) * 64u, sw = static_cast<uint32_t>((r >> 1) & 3);  // 64-byte swizzle
    const uint32_t dst_row = static_cast<uint32_t>((r >> 3) * 256 + (r & 7) * 16);
#pragma unroll 1
    for (int it = g; it < n_items; it += kConvGroups) {
      const int b = it % XB;
      const uint32_t dst = xb0 + static_cast<uint32_t>(b) * (G * kXbBytes) + dst_row;
#pragma unroll
      for (int j = 0; j < G; ++j) {
        const int n = it * G + j;
        if (n >= n_steps) break;
        const int s = n % XF;
        timed_out |= !mbar_wait(xf_full0 + 8u * s, (n / XF) & 1);
        const uint32_t src = xf0 + static_cast<uint32_t>(s) * kXfBytes + src_row;
        const float4 f0 = lds_f32x4(src + ((0u ^ sw) << 4));
        float4 f1 = lds_f32x4(src + ((1u ^ sw) << 4));
        const float4 f2 = lds_f32x4(src + ((2u ^ sw) << 4));
        const float4 f3 = lds_f32x4(src + ((3u ^ sw) << 4));
        if (n % KS == KS - 1) f1 = make_float4(1.f, 1.f, 0.f, 0.f);  // the two ones columns that pick up c1 (the copy filled zeros)
        if (j == 0) timed_out |= !mbar_wait(xb_empty0 + 8u * b, ((it / XB) & 1) ^ 1);  // the MMAs that read this buffer are done
        timed_out = __any_sync(0xFFFFFFFFu, timed_out);  // the warp leaves together
        if (timed_out) break;
        sts_v4(dst + j * kXbBytes, pack_bf16(f0.x, f0.y), pack_bf16(f0.z, f0.w), pack_bf16(f1.x, f1.y), pack_bf16(f1.z, f1.w));
        sts_v4(dst + j * kXbBytes + 128, pack_bf16(f2.x, f2.y), pack_bf16(f2.z, f2.w), pack_bf16(f3.x, f3.y), pack_bf16(f3.z, f3.w));
        __syncwarp();
        if ((tid & 31) == 0) mbar_arrive(xf_empty0 + 8u * s);  // after the stores, which needed the loaded values: the stage has been read
      }
      if (timed_out) break;
      fence_async_smem();
      __syncwarp();
      if ((tid & 31) == 0) mbar_arrive_cluster(lead_xb_full0 + 8u * b);
    }
  } else if (tid < kConvThreads + kEpiThreads) {
    // ---- epilogue warps: warp w of the eight takes lane quarter w % 4 and column half w / 4 --------
    const int q = tid - kConvThreads, half = q / 128;
    const int row = q % 128;  // tile row and tensor-memory lane
    const uint32_t lane_off = static_cast<uint32_t>((row / 32) * 32) << 16;
    const uint32_t acc1 = tmem_base + lane_off + static_cast<uint32_t>(half * (kCH / 2));
    const uint32_t hid = tmem_base + kHidCol + lane_off + static_cast<uint32_t>(half * (kCH / 4));
    const uint32_t acc2 = tmem_base + kAcc2Col + lane_off + static_cast<uint32_t>(half * (kCH / 4));
    const uint32_t cv_addr = smem_u32(sm.cv), c2_addr = cv_addr + 4u * (kCH + 4);
    const uint32_t part_full0 = smem_u32(&sm.part_full[0]);
    for (int kt = 0; kt < my_tiles; ++kt) {
      // layer 1: relu, bf16, back into tensor memory as the A operand of layer 2
      timed_out |= !mbar_wait(acc1_full, static_cast<uint32_t>(kt & 1));
      timed_out = __any_sync(0xFFFFFFFFu, timed_out);
      if (timed_out) break;
      tc_fence_after();
      uint32_t ra[32], rb[32], pk[16];
      {
        tmem_ld32_nowait(acc1, ra);
#pragma unroll
        for (int c0 = 0; c0 < kCH / 2; c0 += 64) {
          tmem_ld_wait();
          tmem_ld32_nowait(acc1 + static_cast<uint32_t>(c0 + 32), rb);
          relu_pack32(ra, pk);
          tmem_st16(hid + static_cast<uint32_t>(c0 / 2), pk);
          tmem_ld_wait();
          if (c0 + 64 < kCH / 2) tmem_ld32_nowait(acc1 + static_cast<uint32_t>(c0 + 64), ra);
          relu_pack32(rb, pk);
          tmem_st16(hid + static_cast<uint32_t>(c0 / 2 + 16), pk);
        }
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if ((tid & 31) == 0) mbar_arrive_cluster(lead_h1_full);
      }
      // layer 2, two passes: pass p, column c of this thread's 64 holds output unit half * 128 + p * 64 + c
      float v = 0.0f;
#pragma unroll 1
      for (int p = 0; p < 2; ++p) {
        timed_out |= !mbar_wait(acc2_full, static_cast<uint32_t>(p));
        timed_out = __any_sync(0xFFFFFFFFu, timed_out);
        if (timed_out) break;
        tc_fence_after();
        tmem_ld32_nowait(acc2, ra);
        tmem_ld32_nowait(acc2 + 32u, rb);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if ((tid & 31) == 0) mbar_arrive_cluster(lead_acc2_free);  // the layer-2 accumulator may be overwritten
        const uint32_t u0 = static_cast<uint32_t>(half * (kCH / 2) + p * (kCH / 4));
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const uint32_t u = u0 + static_cast<uint32_t>(2 * i);
          const uint32_t lo = i < 16 ? ra[2 * i] : rb[2 * i - 32], hi = i < 16 ? ra[2 * i + 1] : rb[2 * i - 31];
          const float x0 = __uint_as_float(lo) + lds_f32(c2_addr + 4u * u), x1 = __uint_as_float(hi) + lds_f32(c2_addr + 4u * u + 4u);
          const uint32_t pr = relu_pack_bf16(__float_as_uint(x0), __float_as_uint(x1));  // h2 rounded to bf16, as the operands of the head are
          v = fmaf(__uint_as_float(pr << 16), lds_f32(cv_addr + 4u * u), v);
          v = fmaf(__uint_as_float(pr & 0xFFFF0000u), lds_f32(cv_addr + 4u * u + 4u), v);
        }
      }
      if (timed_out) break;
      // the two column halves of a row meet in shared memory; the lower half adds cv and stores
      const uint32_t pf = part_full0 + 8u * (kt & 1);
      if (half == 1) {
        sm.part[kt & 1][row] = v;
        __syncwarp();
        if ((tid & 31) == 0) mbar_arrive(pf);
      } else {
        timed_out |= !mbar_wait(pf, static_cast<uint32_t>((kt >> 1) & 1));
        timed_out = __any_sync(0xFFFFFFFFu, timed_out);
        if (timed_out) break;
        v = (v + sm.part[kt & 1][row]) + lds_f32(cv_addr + 4u * kCH);
        const int tile = tile_of(kt);
        const bool in_main = tile < tiles_main;
        const long long r_loc = static_cast<long long>(in_main ? tile : tile - tiles_main) * kTileRows + row;
        if (r_loc < (in_main ? rows_main : rows_total - rows_main)) {
          float *out = values + (in_main ? r_loc : rows_main + r_loc) * N;
#pragma unroll
          for (int n = 0; n < N; ++n) out[n] = v;
        }
      }
    }
  } else if (tid == kConvThreads + kEpiThreads) {
    // ---- the copy thread ----------------------------------------------------------------------
    int n = 0;
    for (int kt = 0; kt < my_tiles && !timed_out; ++kt) {
      // a tile index past the last tile lands past the end of the second array: all zeros
      const int tile = tile_of(kt);
      const bool in_main = tile < tiles_main;
      const CUtensorMap *map = in_main ? &map_main : &map_last;
      const int y = (in_main ? tile : tile - tiles_main) * kTileRows;
      // the next tile's rows are asked into L2 a whole tile ahead, so that the copies above find them there
      const int tile_nx = tile_of(kt + 1);
      const bool nx_main = tile_nx < tiles_main, nx = kt + 1 < my_tiles && tile_nx < n_tiles;
      const CUtensorMap *map_nx = nx_main ? &map_main : &map_last;
      const int y_nx = (nx_main ? tile_nx : tile_nx - tiles_main) * kTileRows;
      for (int ks = 0; ks < KS; ++ks, ++n) {
        if (nx) tma_prefetch_2d(map_nx, ks * 16, y_nx);
        const int s = n % XF;
        timed_out |= !mbar_wait(xf_empty0 + 8u * s, ((n / XF) & 1) ^ 1);
        if (timed_out) break;
        mbar_expect_tx(xf_full0 + 8u * s, kXfBytes);
        tma_load_2d(xf0 + static_cast<uint32_t>(s) * kXfBytes, map, ks * 16, y, xf_full0 + 8u * s);
      }
    }
    if (timed_out)  // let the copies still in flight land before the block goes away
      for (int j = n > XF ? n - XF : 0; j < n; ++j) mbar_wait(xf_full0 + 8u * (j % XF), (j / XF) & 1);
  } else if (tid == kConvThreads + kEpiThreads + 32 && rank == 0) {
    // ---- the MMA-issuing thread of the pair -----------------------------------------------------
    const uint32_t c1_addr = smem_u32(sm.c1), c2_addr = smem_u32(sm.c2);
    const uint32_t acc2_free = smem_u32(&sm.acc2_free), h1_full = smem_u32(&sm.h1_full);
    constexpr uint32_t idesc1 = instr_desc(2 * kTileRows, kCH), idesc2 = instr_desc(2 * kTileRows, kCH / 2);
    uint32_t pass = 0;  // layer-2 passes issued so far; pass j waits for the epilogue of pass j - 1
    // one pass of layer 2: each CTA's output units 64 p .. 64 p + 63 of its half of C2, A = h1 from tensor memory
    auto issue_l2_pass = [&](int p) {
      tc_fence_after();
#pragma unroll
      for (int j = 0; j < kCH / 16; ++j)
        mma2_bf16_ts(tmem_base + kAcc2Col, tmem_base + kHidCol + static_cast<uint32_t>(j * 8),
                     smem_desc(c2_addr + static_cast<uint32_t>(p) * (kCH / 4 / 8) * (kCH * 16) + static_cast<uint32_t>(j) * 256, 128, kCH * 16),
                     idesc2, j > 0 ? 1u : 0u);
      mma2_commit(acc2_full);
      ++pass;
    };
    bool pending = false;  // the second pass of the previous tile is still to be issued
    int n = 0;
    for (int kt = 0; kt < my_tiles && !timed_out; ++kt) {
      for (int ks = 0; ks < KS; ++ks, ++n) {
        if (pending && mbar_try_wait(acc2_free, (pass & 1) ^ 1)) {  // the first pass has been drained: slip the second one in
          issue_l2_pass(1);
          pending = false;
        }
        const int it = n / G, j = n % G, b = it % XB;
        if (j == 0) {
          timed_out |= !mbar_wait(xb_full0 + 8u * b, (it / XB) & 1);
          if (timed_out) break;
          tc_fence_after();
        }
        mma2_bf16(tmem_base, smem_desc(xb0 + static_cast<uint32_t>(b) * (G * kXbBytes) + static_cast<uint32_t>(j) * kXbBytes, 128, 256),
                  smem_desc(c1_addr + static_cast<uint32_t>(ks) * 256, 128, K1 * 16), idesc1, ks > 0 ? 1u : 0u);
        if (j == G - 1 || n == n_steps - 1) mma2_commit(xb_empty0 + 8u * b);  // frees the buffer in both CTAs when its MMAs have read it
      }
      if (timed_out) break;
      if (pending) {  // h1 of the previous tile must have been used up before this tile's replaces it
        timed_out |= !mbar_wait(acc2_free, (pass & 1) ^ 1);
        if (timed_out) break;
        issue_l2_pass(1);
        pending = false;
      }
      mma2_commit(acc1_full);
      timed_out |= !mbar_wait(h1_full, static_cast<uint32_t>(kt & 1));  // relu(h1) of both CTAs is in tensor memory
      if (!timed_out) timed_out |= !mbar_wait(acc2_free, (pass & 1) ^ 1);
      if (timed_out) break;
      issue_l2_pass(0);
      pending = true;
    }
    if (pending && !timed_out) {
      timed_out |= !mbar_wait(acc2_free, (pass & 1) ^ 1);
      if (!timed_out) issue_l2_pass(1);
    }
  }
  if (timed_out) atomicExch(status, kStatusTimeout);
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // neither CTA leaves, or frees tensor memory, while the other may still use it
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

}  // namespace

size_t critic_weight_bytes(const mava_config_t &cfg) {
  return find_variant(cfg) == 3 ? CriticShape<4>::IMAGE_BYTES : 16;
}

cudaError_t launch_critic_tc(mava_rollout *h, const float *params_dev, int32_t T) {
  if (h->variant != 3 || !h->d_critic || !h->d_obs_last) return cudaErrorNotSupported;
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
  CUtensorMap map_main, map_last;
  // boxes of 128 rows x 16 columns (64 bytes, 64-byte swizzle): one K step of one tile
  if (!encode_f32_map(&map_main, h->buf.obs, S::KJ, rows_main, 16, kTileRows, CU_TENSOR_MAP_SWIZZLE_64B) ||
      !encode_f32_map(&map_last, h->d_obs_last, S::KJ, h->cfg.n_envs, 16, kTileRows, CU_TENSOR_MAP_SWIZZLE_64B))
    return cudaErrorInvalidValue;
  const int pair_tiles = (n_tiles + 1) / 2, pairs = pair_tiles < sms / 2 ? pair_tiles : sms / 2;
  auto go = [&](auto kern, size_t smem) {
    smem += 1024;  // room to align the struct by hand
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (err != cudaSuccess) return;
    kern<<<2 * pairs, kCriticThreads, smem, h->stream>>>(map_main, map_last, tiles_main, rows_main, rows_total, image, h->buf.values,
                                                         n_tiles, h->d_status);
    err = cudaGetLastError();
  };
  // six fp32 stages in flight (48 KB per SM), six one-step operand buffers
  go(critic_kernel<4, 6, 6, 1>, sizeof(CriticSmem<4, 6, 6, 1>));
  h->launches += 1;
  return err;
}

}  // namespace mava
