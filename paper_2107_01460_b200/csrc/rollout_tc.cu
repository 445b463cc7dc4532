// bf16 tensor-core rollout for sm_100a: tcgen05.mma with fp32 accumulators in tensor memory.
//
// One persistent CTA per SM keeps the bf16 weights resident in shared memory (loaded once with
// bulk async copies, in the canonical K-major core-matrix layout the MMA reads) and runs one or
// two independent groups of 128 threads.  A group owns one tile of environments (up to 128
// agent rows = the M of the MMA; thread r owns row r and tensor-memory lane r) for all T steps,
// then takes its next tile.  The environment lives in registers (env.cuh).  Per step a group
//   1. writes the non-zero entries of its observation rows into a zeroed bf16 A tile,
//   2. starts layer 1 and, while it runs, sends the observation block to the time-major obs
//      array and draws the Philox uniform of the step,
//   3. runs layer 2 and the heads, each MMA batch issued by one thread and completing on an
//      mbarrier; the epilogues read the accumulators out of tensor memory (ReLU, bf16) and hand
//      the row back as the next A operand; the heads' epilogue is the sampler (softmax,
//      inverse-CDF action, log-prob),
//   4. applies the transition and auto-reset with warp shuffles and ballots.
// Two layouts of the per-step data are compiled:
//   TM = false (H <= 128): the fp32 observation block is staged in shared memory in the global
//     layout (one vectorised contiguous copy) and the hidden activations go back to shared memory;
//   TM = true (H = 256, where the weights leave no room): the hidden activations stay in tensor
//     memory as the A operand of the next MMA and the observation block is expanded from the
//     bf16 A tile on its way out.
// Groups never wait for one another.  Every wait on an mbarrier is bounded: when it runs out the
// group records kStatusTimeout, stops stepping and falls through to the common exit.
#include <cuda_bf16.h>

#include "common.cuh"
#include "env.cuh"
#include "env_wh.cuh"
#include "layout.h"
#include "tc_common.cuh"

namespace mava {
namespace {


// ---- shapes ------------------------------------------------------------------------------------
template <int N, int H, bool TM>
struct TcShape {
  static constexpr int D = kObsFixed + N;
  static constexpr int K1 = (D + 15) / 16 * 16;               // layer-1 K padded to the MMA's K step
  static constexpr int EPW = 32 / N;                           // environments per warp (lanes EPW*N.. idle)
  static constexpr int RPW = EPW * N;                          // agent rows per warp
  static constexpr int EPT_MAX = 4 * EPW;                      // environments per tile, at most
  // With two spare K columns the layer-1 bias rides in W1 (A columns D, D+1 are set to 1).
  static constexpr bool FOLD1 = (K1 - D >= 2);
  // Weight image: W1 | W2 | heads | bias tiles | the constant "ones" A tile.  A bias tile is an
  // N x 16 operand whose column 0 holds bf16(b) and column 1 the bf16 of the remainder; multiplied
  // by the ones tile (columns 0 and 1 equal to 1) it seeds the accumulator with the bias to about
  // 2^-17 relative, so the epilogues need no bias arithmetic.
  static constexpr uint32_t W1_OFF = 0, W1_BYTES = H * K1 * 2;
  static constexpr uint32_t W2_OFF = W1_OFF + W1_BYTES, W2_BYTES = H * H * 2;
  static constexpr uint32_t WH_OFF = W2_OFF + W2_BYTES, WH_BYTES = kHeadRows * H * 2;
  static constexpr uint32_t BT_BYTES = H * 16 * 2;
  static constexpr uint32_t B1_OFF = WH_OFF + WH_BYTES;
  static constexpr uint32_t B2_OFF = B1_OFF + (FOLD1 ? 0 : BT_BYTES);
  static constexpr uint32_t BH_OFF = B2_OFF + BT_BYTES, BH_BYTES = 32;  // 8 floats: ba[0..5], bv, 0
  static constexpr uint32_t ONES_OFF = BH_OFF + BH_BYTES, ONES_BYTES = kTileRows * 16 * 2;
  static constexpr uint32_t IMAGE_BYTES = ONES_OFF + ONES_BYTES;
  static constexpr uint32_t A_BYTES = (kTileRows / 8) * (K1 / 8) * 144;  // padded core-matrix pitch, see a_offset
  static constexpr uint32_t STAGE_BYTES = (kTileRows * D * 4 + 15) / 16 * 16;
  // Tensor-memory columns of one group: accumulator (reused by both hidden layers), the bf16
  // hidden activations (two per column) when TM, the heads accumulator.
  static constexpr int HID_COL = H;
  static constexpr int HEAD_COL = H + (TM ? H / 2 : 0);
  static constexpr int GROUP_COLS = HEAD_COL + 64;  // two heads accumulators: one per thread group in ping-pong mode
  // TM with room for two groups' columns (H <= 128): the fp32 observation block is kept as well and leaves as a bulk
  // copy.  Nothing else lives in its memory, so the copy has a whole step to read it.
  static constexpr bool STG = TM && 2 * GROUP_COLS <= 512;
  static constexpr uint32_t X_BYTES =
      TM ? (STG ? STAGE_BYTES : 16) : (STAGE_BYTES > kTileRows * H * 2 ? STAGE_BYTES : kTileRows * H * 2);
  // independent sets of tile resources (A tile, block, tensor-memory columns) per CTA
  static constexpr int GROUPS = (2 * GROUP_COLS <= 512 && 2 * (A_BYTES + X_BYTES) + IMAGE_BYTES <= 220 * 1024) ? 2 : 1;
  static constexpr int TMEM_COLS = GROUPS * GROUP_COLS <= 256 ? 256 : 512;
  // When only one set of tile resources fits (H = 256), two thread groups still run, in
  // anti-phase: they take turns on the one A tile and on the accumulator and hidden-activation
  // columns of tensor memory (each handed over as soon as its last reader is done), so
  // that one group's environment phase (sampler, transition, observation) overlaps the other's
  // network phase (the three MMAs and their epilogues).
  static constexpr bool PINGPONG = TM && GROUPS == 1;
  // In ping-pong mode a third warpgroup sends the observation blocks out (bf16 A tile -> fp32 rows of the obs array):
  // on the two thread groups' own time that copy was a quarter of the step.
  static constexpr bool HELPERS = PINGPONG;
  static constexpr int THREADS = (HELPERS ? 3 : 2) * kGroupThreads;
  // Registers: the block starts with 65536 / 384 rounded down to a multiple of 8 per thread; the helpers give theirs
  // back (kHelperRegs) and the two groups take kGroupRegs each: 256 * 200 + 128 * 72 = 60416 <= 384 * 160.
  static constexpr int kGroupRegs = 200, kHelperRegs = 72;
};

template <int N, int F, int H, bool TM>
struct TcGroupSmem {
  using S = TcShape<N, H, TM>;
  // TM = false: the fp32 observation block in the global layout while a step starts, the hidden
  // activations (A operand of layer 2 and of the heads) for the rest of the step.
  alignas(128) unsigned char x[S::X_BYTES];
  alignas(128) unsigned char a[S::A_BYTES];  // bf16 observations, A operand of layer 1
  float step_frac[kTileRows];                // exact step/cap of each row (bf16 in A is rounded)
};

template <int N, int F, int H, bool TM>
struct TcSmem {
  using S = TcShape<N, H, TM>;
  alignas(128) unsigned char weights[S::IMAGE_BYTES];
  TcGroupSmem<N, F, H, TM> grp[S::GROUPS];
  alignas(8) uint64_t mma_bar[2];  // one per thread group
  alignas(8) uint64_t load_bar;
  uint32_t tmem_base;
  int abort;  // ping-pong mode: a group gave up; both finish their barrier protocol without work
  int copy_rows[2];  // ping-pong mode, per group: rows of the step's observation block the helpers send out (0: none)
};


template <int N, int H, bool TM, bool CENTRAL>
__global__ void prep_tc_kernel(const float *__restrict__ params, unsigned char *__restrict__ image, ParamLayout L) {
  using S = TcShape<N, H, TM>;
  constexpr int D = S::D, K1 = S::K1;
  auto at = [&](uint32_t off) { return reinterpret_cast<__nv_bfloat16 *>(image + off); };
  const int tid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
  for (int i = tid; i < H * K1; i += nth) {
    const int n = i / K1, k = i - n * K1;
    __nv_bfloat16 v = __float2bfloat16_rn(k < D ? params[L.W1 + static_cast<size_t>(n) * D + k] : 0.0f);
    if (S::FOLD1 && (k == D || k == D + 1)) {
      __nv_bfloat16 hi, lo;
      split_bf16(params[L.b1 + n], hi, lo);
      v = (k == D) ? hi : lo;
    }
    at(S::W1_OFF)[canon_offset(n, k, K1) / 2] = v;
  }
  for (int i = tid; i < H * H; i += nth) {
    const int n = i / H, k = i - n * H;
    at(S::W2_OFF)[canon_offset(n, k, H) / 2] = __float2bfloat16_rn(params[L.W2 + static_cast<size_t>(n) * H + k]);
  }
  for (int i = tid; i < kHeadRows * H; i += nth) {
    const int n = i / H, k = i - n * H;
    float v = 0.0f;
    if (n < kActions) v = params[L.Wa + static_cast<size_t>(n) * H + k];
    else if (n == kActions && !CENTRAL) v = params[L.Wv + k];  // the centralised critic has its own kernels
    at(S::WH_OFF)[canon_offset(n, k, H) / 2] = __float2bfloat16_rn(v);
  }
  // bias tiles of the hidden layers (hi, lo, then zeros), the heads' biases as fp32, the ones tile
  for (int i = tid; i < 2 * H * 16; i += nth) {
    const int r = i / 16, k = i - r * 16;
    float b;
    uint32_t off;
    int n;
    if (r < H) {
      if (S::FOLD1) continue;
      b = params[L.b1 + r]; off = S::B1_OFF; n = r;
    } else {
      b = params[L.b2 + r - H]; off = S::B2_OFF; n = r - H;
    }
    __nv_bfloat16 hi, lo;
    split_bf16(b, hi, lo);
    at(off)[canon_offset(n, k, 16) / 2] = k == 0 ? hi : (k == 1 ? lo : __float2bfloat16_rn(0.0f));
  }
  if (tid < 8)
    reinterpret_cast<float *>(image + S::BH_OFF)[tid] =
        tid < kActions ? params[L.ba + tid] : ((tid == kActions && !CENTRAL) ? params[L.bv] : 0.0f);
  for (int i = tid; i < kTileRows * 16; i += nth) {
    const int r = i / 16, k = i - r * 16;
    at(S::ONES_OFF)[canon_offset(r, k, 16) / 2] = __float2bfloat16_rn(k < 2 ? 1.0f : 0.0f);
  }
}


// Epilogue of a hidden layer: thread `row` reads its accumulator row (bias already inside) from
// tensor memory, applies ReLU and rounds to bf16; the row becomes the A operand of the next
// layer, either in shared memory (canonical layout, K = H) or, packed two per column, in tensor
// memory.  The load of the next 32 columns is in flight while the current 32 are converted.
template <int H, bool TM>
__device__ __forceinline__ void hidden_epilogue(uint32_t acc_taddr, uint32_t hid_taddr, uint32_t hbuf, int row) {
  static_assert(H % 64 == 0, "two 32-column batches per iteration");
  uint32_t ra[32], rb[32], pk[16];
  tmem_ld32_nowait(acc_taddr, ra);
#pragma unroll
  for (int c0 = 0; c0 < H; c0 += 64) {
    tmem_ld_wait();
    tmem_ld32_nowait(acc_taddr + static_cast<uint32_t>(c0 + 32), rb);
    relu_pack32(ra, pk);
    if (TM) {
      tmem_st16(hid_taddr + static_cast<uint32_t>(c0 / 2), pk);
    } else {
#pragma unroll
      for (int q = 0; q < 4; ++q)
        sts_v4(hbuf + canon_offset(row, c0 + 8 * q, H), pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
    }
    tmem_ld_wait();
    if (c0 + 64 < H) tmem_ld32_nowait(acc_taddr + static_cast<uint32_t>(c0 + 64), ra);
    relu_pack32(rb, pk);
    if (TM) {
      tmem_st16(hid_taddr + static_cast<uint32_t>(c0 / 2 + 16), pk);
    } else {
#pragma unroll
      for (int q = 0; q < 4; ++q)
        sts_v4(hbuf + canon_offset(row, c0 + 32 + 8 * q, H), pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
    }
  }
  if (TM) tmem_st_wait();
}


// One dense layer on the tensor core, issued by a single thread: the accumulator is seeded with
// the bias (ones tile x bias tile, K = 16) unless the bias rides in the weights, and then
// accumulates K / 16 steps of A x W^T, A from shared memory or from tensor memory.
template <int K, int NOUT, bool BIAS_TILE, bool A_TMEM, uint32_t A_LBO = 128>
__device__ __forceinline__ void issue_layer(uint32_t d_tmem, uint32_t a_addr, uint32_t w_addr, uint32_t ones_addr,
                                            uint32_t bias_addr, uint32_t bar) {
  constexpr uint32_t idesc = instr_desc(kTileRows, NOUT);
  if (BIAS_TILE) mma_bf16(d_tmem, smem_desc(ones_addr, 128, 256), smem_desc(bias_addr, 128, 256), idesc, 0);
#pragma unroll
  for (int k = 0; k < K / 16; ++k) {
    const uint32_t acc = (BIAS_TILE || k > 0) ? 1u : 0u;
    if (A_TMEM) mma_bf16_ts(d_tmem, a_addr + k * 8, smem_desc(w_addr + k * 256, 128, K * 16), idesc, acc);
    else
      mma_bf16(d_tmem, smem_desc(a_addr + k * 2 * A_LBO, A_LBO, (K / 8) * A_LBO), smem_desc(w_addr + k * 256, 128, K * 16),
               idesc, acc);
  }
  mma_commit(bar);
}

// Observation rows [first, first + n) of a tile (compact numbering; tile row = tile_row0 + i),
// expanded from the bf16 A tile to fp32 and written to `dst` (row stride D); consecutive lanes
// write consecutive floats.  The exact step/cap replaces the rounded bf16 one.  Four rows are in
// flight at a time.
template <int D, int K1>
__device__ __forceinline__ void expand_rows(uint32_t a_tile, uint32_t step_frac, float *dst, int first, int n,
                                            int tile_row0, int lane) {
  constexpr int Q = (D + 31) / 32;
  uint32_t off[Q];
#pragma unroll
  for (int q = 0; q < Q; ++q) off[q] = a_offset<K1>(0, lane + 32 * q);
  for (int l0 = 0; l0 < n; l0 += 4) {
    uint32_t raw[4][Q];
    float sf[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int tr = tile_row0 + min(l0 + r, n - 1);
      const uint32_t arow = a_tile + a_offset<K1>(tr, 0);
#pragma unroll
      for (int q = 0; q < Q; ++q) raw[r][q] = (lane + 32 * q < D) ? lds_u16(arow + off[q]) : 0u;
      sf[r] = lds_f32(step_frac + 4u * static_cast<uint32_t>(tr));
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      if (l0 + r < n) {
        float *orow = dst + static_cast<size_t>(first + l0 + r) * D;
#pragma unroll
        for (int q = 0; q < Q; ++q) {
          const int j = lane + 32 * q;
          if (j < D) orow[j] = (j == 3 * kPlane + 1) ? sf[r] : __uint_as_float(raw[r][q] << 16);
        }
      }
    }
  }
}

// The same job for row counts that are multiples of four: four rows are one 16-byte aligned run
// of 4*D floats, written as float4 by consecutive lanes.  Which (row of the four, column) a lane's
// elements are does not depend on the quad, so their tile offsets are computed once.
template <int D, int K1>
struct QuadPlan {
  static constexpr int V = (D + 31) / 32;  // float4 per lane per quad (D float4 in all)
  uint32_t off[V][4];                      // byte offset inside the A tile relative to the quad's first row
  uint32_t frac_row[V];                    // row (0..3) whose step/cap this lane's float4 may contain
  bool is_frac[V][4];                      // element i of float4 v is a step/cap entry
};
template <int D, int K1>
__device__ __forceinline__ void plan_quads(QuadPlan<D, K1> &p, int lane) {
#pragma unroll
  for (int v = 0; v < QuadPlan<D, K1>::V; ++v) {
    p.frac_row[v] = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int f = 4 * (lane + 32 * v) + i;  // float index inside the quad (< 4*D when the lane takes part)
      const int r = f / D, j = f - r * D;
      p.off[v][i] = a_offset<K1>(r & 3, j);   // a quad starts at a multiple of four rows: no carry into the 8-row group
      p.is_frac[v][i] = (j == 3 * kPlane + 1 && r < 4);
      if (p.is_frac[v][i]) p.frac_row[v] = r;
    }
  }
}
// All loads of a quad are issued before the first use, so only one shared-memory latency is paid.
template <int D, int K1>
__device__ __forceinline__ void expand_quads(const QuadPlan<D, K1> &p, uint32_t a_tile, uint32_t step_frac, float *dst,
                                             int first, int n, int tile_row0, int lane) {
  constexpr int V = QuadPlan<D, K1>::V;
  constexpr int U = 2;  // quads in flight
  for (int l0 = 0; l0 < n; l0 += 4 * U) {
    uint32_t raw[U][V][4];
    float sf[U][V];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int tr = tile_row0 + min(l0 + 4 * u, n - 4);
      const uint32_t qbase = a_tile + a_offset<K1>(tr, 0);
#pragma unroll
      for (int v = 0; v < V; ++v) {
#pragma unroll
        for (int i = 0; i < 4; ++i) raw[u][v][i] = (lane + 32 * v < D) ? lds_u16(qbase + p.off[v][i]) : 0u;
        sf[u][v] = lds_f32(step_frac + 4u * (static_cast<uint32_t>(tr) + p.frac_row[v]));
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (l0 + 4 * u < n) {
        float4 *out = reinterpret_cast<float4 *>(dst + static_cast<size_t>(first + l0 + 4 * u) * D);
#pragma unroll
        for (int v = 0; v < V; ++v) {
          if (lane + 32 * v < D) {
            float e[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) e[i] = p.is_frac[v][i] ? sf[u][v] : __uint_as_float(raw[u][v][i] << 16);
            out[lane + 32 * v] = make_float4(e[0], e[1], e[2], e[3]);
          }
        }
      }
    }
  }
}

// ---- the rollout kernel ------------------------------------------------------------------------
template <int N, int F, int H, bool TM, bool EVAL, int ENV = 0>
__global__ void __launch_bounds__(TcShape<N, H, TM>::THREADS, 1)
rollout_tc_kernel(RolloutArgs a, const unsigned char *__restrict__ image, int ept, int n_tiles, int groups) {
  using S = TcShape<N, H, TM>;
  constexpr int D = S::D, K1 = S::K1;
  constexpr bool PP = S::PINGPONG;
  constexpr bool HP = S::HELPERS;       // the third warpgroup sends the observation blocks out
  constexpr int TP = HP ? 3 : 2;        // parties of the A tile's hand-over barrier
  extern __shared__ __align__(128) unsigned char smem_raw[];
  TcSmem<N, F, H, TM> &sm = *reinterpret_cast<TcSmem<N, F, H, TM> *>(smem_raw);
  const int tid = threadIdx.x;
  const bool helper = HP && tid >= 2 * kGroupThreads;
  const int g = helper ? 0 : tid / kGroupThreads;   // thread group
  const int dg = PP ? 0 : g;           // the set of tile resources it uses
  const int row = tid % kGroupThreads; // row of the tile this thread owns; also its TMEM lane
  const int warp = tid / 32, lane = tid & 31;
  const int wg = row / 32;             // warp inside the group
  TcGroupSmem<N, F, H, TM> &gs = sm.grp[dg];

  // ---- one-time set-up: barriers, tensor memory, weights -------------------------------------
  if (tid == 0) {
    sm.abort = 0;
    mbar_init(smem_u32(&sm.load_bar), 1);
    mbar_init(smem_u32(&sm.mma_bar[0]), 1);
    mbar_init(smem_u32(&sm.mma_bar[1]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                 "r"(S::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if ((!PP || g == 0) && !helper) {  // zero the observation block and the A operand once
    uint4 *z = reinterpret_cast<uint4 *>(gs.x);
    for (int i = row; i < static_cast<int>(S::X_BYTES / 16); i += kGroupThreads) z[i] = make_uint4(0, 0, 0, 0);
    z = reinterpret_cast<uint4 *>(gs.a);
    for (int i = row; i < static_cast<int>(S::A_BYTES / 16); i += kGroupThreads) z[i] = make_uint4(0, 0, 0, 0);
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
  timed_out = __syncthreads_or(timed_out) != 0;  // uniform: the loops below depend on it

  const uint32_t tmem_base = sm.tmem_base;
  const uint32_t acc_col = tmem_base + static_cast<uint32_t>(dg * S::GROUP_COLS);
  const uint32_t hid_col = acc_col + static_cast<uint32_t>(S::HID_COL);
  const uint32_t head_col = acc_col + static_cast<uint32_t>(S::HEAD_COL + (PP ? 32 * g : 0));
  const uint32_t lane_off = static_cast<uint32_t>(wg * 32) << 16;  // this warp's TMEM lanes
  const uint32_t w_addr = smem_u32(sm.weights);
  const uint32_t a_addr = smem_u32(gs.a);
  const uint32_t frac_addr = smem_u32(gs.step_frac), stage_addr = smem_u32(gs.x), abort_addr = smem_u32(&sm.abort);
  const uint32_t h_addr = TM ? hid_col : smem_u32(gs.x);  // A operand of layer 2 and of the heads
  const uint32_t bar = smem_u32(&sm.mma_bar[g]);
  const float *head_bias = reinterpret_cast<const float *>(sm.weights + S::BH_OFF);
  float *stage = reinterpret_cast<float *>(gs.x);
  uint32_t phase = 0;
  bool bulk_pending = false;  // thread 0 of a group: a bulk store of the observation block is in flight
  const size_t M = static_cast<size_t>(a.env.n_envs) * N;
  const int le = wg * S::EPW + lane / N;  // local environment of this lane
  const int ag = lane % N;                // its agent
  const int crow = le * N + ag;           // compact row inside the tile's block

  if (helper) {
    if constexpr (HP) {
      // ---- helper warpgroup: for every step of either group, in the order in which the groups use the A tile, wait
      // until the step's observations are in the tile, expand the rows the group asks for to fp32 in the obs array
      // (warp w the rows of the group's warp w), and let go of the tile.  The loop bounds are those of the groups,
      // which in ping-pong mode walk through every step's barriers whatever happens to them.
      asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(S::kHelperRegs));
      QuadPlan<D, K1> quad_plan;
      if (N % 4 == 0) plan_quads<D, K1>(quad_plan, lane);
      pair_arrive(kBarTile + 0, TP);  // group 0 goes first
      const volatile int *copy_rows = sm.copy_rows;
      for (int it = 0;; ++it) {
        const int tile0 = (it * static_cast<int>(gridDim.x) + static_cast<int>(blockIdx.x)) * groups;
        if (tile0 >= n_tiles) break;
        for (int t = 0; t <= (EVAL ? a.T - 1 : a.T); ++t) {
          for (int hg = 0; hg < 2; ++hg) {
            pair_sync(kBarReady + hg);
            const int n_rows = copy_rows[hg];
            if (n_rows > 0) {
              const int e0 = (tile0 + hg) * ept;
              float *dst = (t == a.T) ? a.obs_last + static_cast<size_t>(e0) * N * D
                                      : a.buf.obs + (static_cast<size_t>(t) * M + static_cast<size_t>(e0) * N) * D;
              if constexpr (N % 4 == 0)
                expand_quads<D, K1>(quad_plan, a_addr, frac_addr, dst, wg * S::RPW, min(S::RPW, n_rows - wg * S::RPW), wg * 32, lane);
              else
                expand_rows<D, K1>(a_addr, frac_addr, dst, wg * S::RPW, min(S::RPW, n_rows - wg * S::RPW), wg * 32, lane);
            }
            pair_arrive(kBarTile + (1 - hg), TP);
          }
        }
      }
    }
  } else {
  // ---- the two thread groups (everything up to the common exit) ------------------------------------------------
  if constexpr (HP) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(S::kGroupRegs));
  QuadPlan<D, K1> quad_plan;
  if (PP && !HP && N % 4 == 0) plan_quads<D, K1>(quad_plan, lane);
  if (PP && g == 1) {  // group 0 goes first on both shared resources
    pair_arrive(kBarTile + 0, TP);
    pair_arrive(kBarTmem + 0);
    pair_arrive(kBarHid + 0);
  }

  // ---- tiles: in round `it` group g works on tile (it * gridDim.x + blockIdx.x) * groups + g; with
  // groups == 1 (little work: one group per SM has the tensor pipe to itself) group 1 sits out ------
  for (int it = 0; !timed_out || PP; ++it) {
    const int tile0 = (it * static_cast<int>(gridDim.x) + static_cast<int>(blockIdx.x)) * groups;
    if (tile0 >= n_tiles) break;  // same for both groups
    const int tile = tile0 + g;
    if (!PP && (g >= groups || tile >= n_tiles)) break;
    // ping-pong: a group without a tile (or after a time-out) still walks through the hand-over
    // barriers of every step, so that its partner never waits for it in vain
    bool idle = PP && (tile >= n_tiles || timed_out);
    const int e0 = tile * ept;
    const int n_env = idle ? 0 : min(ept, a.env.n_envs - e0);
    const int n_rows = n_env * N;
    const bool active = lane < S::RPW && le < n_env;
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

    // Per-row outputs of a step wait in registers and go to global memory while the next step's
    // layer 1 runs: a named barrier also waits for the stores issued before it, so stores placed
    // right before one would put their round trip to L2 on the critical path.
    bool pend = false, pend_step = false, pend_done = false;
    size_t pend_row0 = 0, pend_done_idx = 0;
    float pend_value = 0.0f, pend_logp = 0.0f, pend_reward = 0.0f, pend_logit[kActions];
    int pend_action = 0;
#pragma unroll
    for (int k = 0; k < kActions; ++k) pend_logit[k] = 0.0f;
    auto flush_outputs = [&]() {
      if (pend && active) {
        a.buf.values[pend_row0 + crow] = pend_value;
        if (pend_step) {
          a.buf.actions[pend_row0 + crow] = pend_action;
          a.buf.logp[pend_row0 + crow] = pend_logp;
          a.buf.rewards[pend_row0 + crow] = pend_reward;
          if (ag == 0) a.buf.dones[pend_done_idx] = pend_done ? 1 : 0;
          if (a.write_logits) {
#pragma unroll
            for (int k = 0; k < kActions; ++k) a.buf.logits[(pend_row0 + crow) * kActions + k] = pend_logit[k];
          }
        }
      }
      pend = false;
    };
    constexpr bool ev = EVAL;     // evaluation block: nothing of the trajectory is stored
    EvalSums sums;                // lanes with ag == 0: their environment
    for (int t = 0; t <= (ev ? a.T - 1 : a.T); ++t) {
      const bool last = !ev && (t == a.T);
      const size_t row0 = static_cast<size_t>(t) * M + static_cast<size_t>(e0) * N;
      if (PP) {
        pair_sync(kBarTile + g, TP);  // the other group (and the helpers' copy of its rows) is done with the A tile
        // one decision for the whole group (its threads may see the flag at different times); the flag
        // is looked at every eighth step only: the load would queue behind the partner's copy-out
        idle = group_any(g, idle || ((t & 7) == 0 && lds_s32(abort_addr) != 0));
        if (idle) {  // keep the hand-over order of a working step: three acquisitions, then three releases
          if (HP) {    // nothing for the helpers to copy
            if (row == 0) *reinterpret_cast<volatile int *>(&sm.copy_rows[g]) = 0;
            pair_arrive(kBarReady + g);
          }
          pair_sync(kBarTmem + g);
          pair_sync(kBarHid + g);
          pair_arrive(kBarTile + (1 - g), TP);
          pair_arrive(kBarTmem + (1 - g));
          pair_arrive(kBarHid + (1 - g));
          continue;
        }
#pragma unroll
        for (int kc = 0; kc < K1 / 8; ++kc)
          sts_zero16(a_addr + a_offset<K1>(row, kc * 8));
      }
      // 1. non-zero observation entries into the zeroed A tile (and the zeroed fp32 block)
      if (active) {
        const uint32_t a_row = a_addr + a_offset<K1>(row, 0);
        auto put = [&](int j, float v) {
          if (!TM || S::STG) sts_f32(stage_addr + 4u * static_cast<uint32_t>(crow * D + j), v);
          else if (j == 3 * kPlane + 1) sts_f32(frac_addr + 4u * static_cast<uint32_t>(row), v);
          sts_u16(a_row + a_offset<K1>(0, j), bf16_bits(v));
        };
        if constexpr (ENV == 0) observe_env<N, F>(env, a.env, ag, put);
        else wh_observe_env<N, F>(env, a.env, ag, put);
        if (S::FOLD1) {  // the two columns that pick up the bias rows of W1
          sts_u16(a_row + a_offset<K1>(0, D), 0x3F80);
          sts_u16(a_row + a_offset<K1>(0, D + 1), 0x3F80);
        }
      }
      if (HP) {  // the helpers take the rows from here (the observation after the last step feeds a centralised critic)
        if (row == 0)
          *reinterpret_cast<volatile int *>(&sm.copy_rows[g]) = (!EVAL && (t < a.T || a.obs_last != nullptr)) ? n_rows : 0;
        __threadfence_block();
        pair_arrive(kBarReady + g);
      }
      fence_async_smem();
      tc_fence_before();
      group_sync(g);
      if (PP) pair_sync(kBarTmem + g);  // the other group's second epilogue has read the accumulator columns
      // 2. layer 1 runs while the previous step's per-row outputs and (when the block is not needed
      //    later) the observation block go to global memory
      if (row == 0) {
        tc_fence_after();
        issue_layer<K1, H, !S::FOLD1, false, kALbo>(acc_col, a_addr, w_addr + S::W1_OFF, w_addr + S::ONES_OFF,
                                             w_addr + S::B1_OFF, bar);
      }
      flush_outputs();  // the previous step's rows
      float *obs_dst = a.buf.obs + row0 * D;
      if (!last && !PP && !ev) {
        if (!TM || S::STG) {  // one contiguous piece of the time-major array
          // by the bulk-copy engine when alignment allows: it leaves the load/store pipe to the
          // other group; the block was fenced for the async proxy together with the A tile
          const int count = n_rows * D;
          if (((row0 * D) & 3) == 0 && (count & 3) == 0) {
            if (row == 0) {
              bulk_store(obs_dst, smem_u32(stage), static_cast<uint32_t>(count) * 4u);
              bulk_pending = true;
            }
          } else {
            for (int i = row; i < count; i += kGroupThreads) obs_dst[i] = stage[i];
          }
        } else {  // this warp's rows, expanded from the bf16 tile
          expand_rows<D, K1>(a_addr, frac_addr, obs_dst, wg * S::RPW, min(S::RPW, n_rows - wg * S::RPW), wg * 32, lane);
          __syncwarp();
        }
      }
      timed_out |= !mbar_wait(bar, phase);
      phase ^= 1;
      if (!TM) {  // every read of the block is done before the epilogue reuses its memory
        if (bulk_pending) { bulk_store_wait_read(); bulk_pending = false; }
        group_sync(g);
      }
      if (HP) pair_arrive(kBarTile + (1 - g), TP);  // layer 1 has read the A tile; the helpers let go of it on their own
      if (PP) pair_sync(kBarHid + g);  // the other group's heads MMA has read the hidden-activation columns
      tc_fence_after();
      hidden_epilogue<H, TM>(acc_col + lane_off, hid_col + lane_off, stage_addr, row);
      if (!TM) fence_async_smem();  // the hidden activations just written feed the next MMA
      tc_fence_before();
      group_sync(g);
      // 3. layer 2; in ping-pong mode its (long) run time hides the observation block's way out
      if (row == 0) {
        tc_fence_after();
        issue_layer<H, H, true, TM>(acc_col, h_addr, w_addr + S::W2_OFF, w_addr + S::ONES_OFF, w_addr + S::B2_OFF, bar);
      }
      // while layer 2 runs: the uniform of this step's action draw, and the A tile (layer 1 is done
      // with it) is zeroed for the next step (ping-pong: the next user of the tile does that)
      float u = 0.0f;
      if (active && !last) u = action_uniform(a.env, a.t_global0 + static_cast<uint32_t>(t), env_id, static_cast<uint32_t>(ag));
      if (TM && !PP) {  // own row only, its readers are in this warp
#pragma unroll
        for (int kc = 0; kc < K1 / 8; ++kc)
          sts_zero16(a_addr + a_offset<K1>(row, kc * 8));
      } else if (!TM) {
        for (int i = row; i < static_cast<int>(S::A_BYTES / 16); i += kGroupThreads) sts_zero16(a_addr + 16u * i);
      }
      if (PP && !HP) {
        if (!ev && (!last || a.obs_last != nullptr)) {  // the observation after the last step feeds a centralised critic
          float *dst = last ? a.obs_last + static_cast<size_t>(e0) * N * D : obs_dst;
          if constexpr (N % 4 == 0)
            expand_quads<D, K1>(quad_plan, a_addr, frac_addr, dst, wg * S::RPW, min(S::RPW, n_rows - wg * S::RPW), wg * 32,
                                lane);
          else
            expand_rows<D, K1>(a_addr, frac_addr, dst, wg * S::RPW, min(S::RPW, n_rows - wg * S::RPW), wg * 32, lane);
        }
        pair_arrive(kBarTile + (1 - g));  // this thread no longer needs the A tile
      }
      timed_out |= !mbar_wait(bar, phase);
      phase ^= 1;
      tc_fence_after();
      hidden_epilogue<H, TM>(acc_col + lane_off, hid_col + lane_off, stage_addr, row);
      if (!TM) fence_async_smem();
      tc_fence_before();
      if (PP) pair_arrive(kBarTmem + (1 - g));  // this thread is done with the accumulator columns
      if (S::STG && bulk_pending) { bulk_store_wait_read(); bulk_pending = false; }  // the block is zeroed after this barrier
      group_sync(g);
      // 4. heads: six logits and the value, N padded to 16
      if (row == 0) {
        tc_fence_after();
        issue_layer<H, kHeadRows, false, TM>(head_col, h_addr, w_addr + S::WH_OFF, 0u, 0u, bar);
      }
      if (S::STG)  // while the heads run: zero the observation block for the next step (its copy has read it)
        for (int i = row; i < static_cast<int>(S::STAGE_BYTES / 16); i += kGroupThreads) sts_zero16(stage_addr + 16u * i);
      timed_out |= !mbar_wait(bar, phase);
      phase ^= 1;
      if (PP) pair_arrive(kBarHid + (1 - g));  // the heads MMA is done reading the hidden-activation columns
      // self-test of the give-up path: nothing of this group is outstanding here, and nothing will complete the
      // barrier's next phase before this group's own next MMA batch
      if (a.debug_expire && blockIdx.x == 0 && g == 0 && it == 0 && t == 1) timed_out |= !mbar_wait(bar, phase, 1u << 12);
      tc_fence_after();
      int action = 0;
      {
        float hv[16];
        tmem_ld16(head_col + lane_off, hv);
#pragma unroll
        for (int k = 0; k <= kActions; ++k) hv[k] += head_bias[k];  // the heads' biases stay fp32
        if (!TM)  // the hidden activations are dead: zero the observation block for the next step
          for (int i = row; i < static_cast<int>(S::STAGE_BYTES / 16); i += kGroupThreads) sts_zero16(stage_addr + 16u * i);
        if (active) {
          pend = !ev; pend_step = !last; pend_row0 = row0; pend_value = hv[kActions];
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
            if (ev) {
              if (a.greedy) action = greedy_action(hv);
              if (a.ev_actions) a.ev_actions[row0 + crow] = action;
            }
            float la = hv[0];
#pragma unroll
            for (int k = 1; k < kActions; ++k) la = (action == k) ? hv[k] : la;
            pend_action = action;
            pend_logp = la - m - __logf(sum);
#pragma unroll
            for (int k = 0; k < kActions; ++k) pend_logit[k] = hv[k];
          }
        }
      }
      tc_fence_before();
      if (group_any(g, timed_out)) {
        timed_out = true;
        if (!PP) break;
        if (row == 0) *reinterpret_cast<volatile int *>(&sm.abort) = 1;  // both groups go idle from their next step on
        idle = true;
        continue;
      }
      if (last) break;
      // 5. transition and auto-reset, inside the warp
      float reward;
      bool done;
      if constexpr (ENV == 0) step_env_warp<N, F>(env, a.env, env_id, ag, base, active, action, reward, done);
      else wh_step_env_warp<N, F>(env, a.env, env_id, base, active, action, reward, done);
      pend_reward = reward;
      pend_done = done;
      pend_done_idx = static_cast<size_t>(t) * a.env.n_envs + e0 + le;
      if (ev) sums.step(reward, done);
    }
    flush_outputs();  // the last step's rows (the bootstrap values among them)
    if (!timed_out && active && ag == 0) {
      store_env(env, a.state[e0 + le]);
      if (ev) { a.ev_count[e0 + le] = sums.count; a.ev_ret[e0 + le] = sums.ret; a.ev_len[e0 + le] = sums.len; }
    }
  }
  if (timed_out && row == 0) atomicExch(a.status, kStatusTimeout);
  }  // thread groups

  bulk_store_wait_all();  // bulk stores of this thread, if any, have landed
  // ---- common exit: every thread arrives here; tensor memory is returned ----------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(S::TMEM_COLS) : "memory");
  }
}

#include "rollout_tc_small.cuh"

// Rows per tile of the few-rows form that serves this batch (0: the 128-row kernel).
template <int N, int H, bool TM>
int few_rows_tile(const mava_rollout *h, int sms) {
  if constexpr (!TM && H == kTileRows) {
    if ((h->cfg.flags & (MAVA_FLAG_WIDE_TILES | MAVA_FLAG_HIDDEN_IN_TMEM)) == 0) {  // either flag asks for the 128-row kernel
      if (h->cfg.n_envs <= sms * SmallShape<N, H, 16>::EPT_MAX) return 16;
      if (h->cfg.n_envs <= sms * SmallShape<N, H, 32>::EPT_MAX) return 32;
    }
  }
  return 0;
}

template <int N, int F, int H, bool TM, int ENV = 0>
cudaError_t launch_tc_variant(mava_rollout *h, const RolloutArgs &args) {
  using S = TcShape<N, H, TM>;
  int sms = 0;
  cudaError_t err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->device);
  if (err != cudaSuccess) return err;
  // Few rows per SM: the form with the rows as the N operand of the MMA.
  if constexpr (H == kTileRows && ENV == 0) {
    const int rb = few_rows_tile<N, H, false>(h, sms);
    if (rb == 16) return launch_tc_small<N, F, H, 16>(h, args, sms);
    if (rb == 32) return launch_tc_small<N, F, H, 32>(h, args, sms);
  }
  auto kern = args.eval ? rollout_tc_kernel<N, F, H, TM, true, ENV> : rollout_tc_kernel<N, F, H, TM, false, ENV>;
  const size_t smem = sizeof(TcSmem<N, F, H, TM>);
  err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (err != cudaSuccess) return err;
  // Environments per tile: full tiles when there is enough work for every group of every SM,
  // otherwise smaller tiles so that all groups have one (the per-step chain is latency-bound).
  // Two thread groups per CTA, unless one group per SM already holds all environments: alone on
  // its SM a group does not share the tensor pipe and the barriers' issue slots.
  const int groups = (!S::PINGPONG && h->cfg.n_envs <= sms * S::EPT_MAX) ? 1 : 2;
  const int slots = sms * groups;
  int ept = (h->cfg.n_envs + slots - 1) / slots;
  if (ept > S::EPT_MAX) ept = S::EPT_MAX;
  if (ept < 1) ept = 1;
  if (!TM || S::STG) {  // tiles whose observation block is a whole number of 16-byte pieces leave as one bulk copy
    for (int e = ept; e <= S::EPT_MAX; ++e)
      if ((e * N * S::D) % 4 == 0) { ept = e; break; }
  }
  const int n_tiles = (h->cfg.n_envs + ept - 1) / ept;
  const int ctas = (n_tiles + groups - 1) / groups;
  kern<<<ctas < sms ? ctas : sms, S::THREADS, smem, h->stream>>>(args, static_cast<const unsigned char *>(h->d_wtc), ept,
                                                                 n_tiles, groups);
  h->launches += 1;
  return cudaGetLastError();
}

template <int N, int H, bool TM, bool CENTRAL = false>
cudaError_t launch_prep_variant(mava_rollout *h, const float *params_dev) {
  prep_tc_kernel<N, H, TM, CENTRAL><<<64, 256, 0, h->stream>>>(params_dev, static_cast<unsigned char *>(h->d_wtc),
                                                     param_layout(h->cfg, h->D, 1));
  h->launches += 1;
  return cudaGetLastError();
}

}  // namespace

// All compiled shapes run on the tensor cores (the centralised critic through critic_tc.cu).
bool tc_supported(const mava_config_t &cfg) {
  const int v = find_variant(cfg);
  return v == 0 || v == 1 || v == 2 || v == 3 || v == 4 || v == 5 || v == 6;
}

// Hidden activations in tensor memory: always for H >= 128 (at H = 128 the fp32 observation block keeps its shared
// memory to itself and its bulk copy has a whole step to read it: 6 % faster than sharing that memory with the
// activations); at H = 64 only when the handle asks for it (MAVA_FLAG_HIDDEN_IN_TMEM), which keeps both layouts
// of the 128-row kernel in use.
static bool use_tm(const mava_rollout *h) {
  return h->cfg.hidden >= 128 || (h->cfg.flags & MAVA_FLAG_HIDDEN_IN_TMEM) != 0;
}

bool tc_rollout_is_wide(const mava_rollout *h) {
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->device) != cudaSuccess) return false;
  if (h->cfg.env_kind != 0 || (h->cfg.flags & MAVA_FLAG_HIDDEN_IN_TMEM) != 0) return true;
  if (h->variant == 1) return few_rows_tile<2, 128, false>(h, sms) == 0;
  if (h->variant == 2) return few_rows_tile<3, 128, false>(h, sms) == 0;
  return true;
}

size_t tc_weight_bytes(const mava_config_t &cfg, int) {
  switch (find_variant(cfg)) {  // the two layouts of a shape have the same image size
    case 0: return TcShape<2, 64, false>::IMAGE_BYTES;
    case 1: return TcShape<2, 128, false>::IMAGE_BYTES;
    case 2: return TcShape<3, 128, false>::IMAGE_BYTES;
    case 3: return TcShape<4, 256, true>::IMAGE_BYTES;
    case 4: return TcShape<8, 256, true>::IMAGE_BYTES;
    case 5: case 6: return rec_tc_weight_bytes(cfg);
    default: return 16;
  }
}

cudaError_t launch_prep_tc(mava_rollout *h, const float *params_dev) {
  switch (h->variant) {
    case 0: return launch_prep_variant<2, 64, false>(h, params_dev);
    case 1: return launch_prep_variant<2, 128, false>(h, params_dev);
    case 2: return launch_prep_variant<3, 128, false>(h, params_dev);
    case 3: return launch_prep_variant<4, 256, true, true>(h, params_dev);
    case 4: return launch_prep_variant<8, 256, true>(h, params_dev);
    default: return cudaErrorNotSupported;
  }
}

cudaError_t launch_rollout_tc(mava_rollout *h, const RolloutArgs &args) {
  const bool tm = use_tm(h);
  if (h->cfg.env_kind != 0) {  // the warehouse family: two shapes
    switch (h->variant) {
      case 0: return launch_tc_variant<2, 2, 64, false, 1>(h, args);
      case 2: return launch_tc_variant<3, 3, 128, true, 1>(h, args);
      default: return cudaErrorNotSupported;
    }
  }
  switch (h->variant) {
    case 0: return tm ? launch_tc_variant<2, 2, 64, true>(h, args) : launch_tc_variant<2, 2, 64, false>(h, args);
    case 1: return launch_tc_variant<2, 2, 128, true>(h, args);
    case 2: return launch_tc_variant<3, 3, 128, true>(h, args);
    case 3: return launch_tc_variant<4, 5, 256, true>(h, args);
    case 4: return launch_tc_variant<8, 8, 256, true>(h, args);
    default: return cudaErrorNotSupported;
  }
}

}  // namespace mava
