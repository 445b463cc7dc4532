// Small-batch form of the bf16 tensor-core rollout (H = 128), included by rollout_tc.cu.
//
// When one SM gets at most RB = 16 or 32 agent rows, a 128-row tile would spend its MMAs and
// epilogues on empty rows while the per-step chain (three dependent MMA round trips) is all that
// counts.  Here the operands change places: the weights are the M = 128 operand (one hidden unit
// per tensor-memory lane), the tile's rows are the N = RB operand, so a K step of 16 costs RB / 2
// instead of 64 tensor-pipe cycles and an epilogue handles RB instead of 128 columns per thread.
// The products and their order of accumulation (bias tile first, then K in ascending steps) are
// those of the 128-row kernel, and so are the results.
//   thread j of the CTA: hidden unit j in the epilogues (tensor-memory lane j);
//   threads 0 .. RB-1 (warp 0): also agent row j of the tile: sampler, transition, level planes of
//   the observation; after a transition they publish their cell, level and step count in shared
//   memory, from which lane j of warp 1 writes row j's wall plane and lane j of warp 2 its scalars
//   (this serial code is bound by instruction latency, so three warps finish it sooner than one).
// Same weight image as the 128-row kernel; the heads (16 rows there) are copied into a zero-padded
// 64-row operand once per CTA.
#pragma once

// The heads are an M = 64 operand (the smallest M): their seven rows come out in lanes 0..6; the
// time of an MMA here is the time to stream its M operand from shared memory.
constexpr int kHeadM = 64;

template <int N, int H, int RB>
struct SmallShape {
  using S = TcShape<N, H, false>;
  static_assert(H == kTileRows, "the hidden width is the M of the MMA");
  static_assert(RB == 16 || RB == 32, "rows per tile: one tensor-memory load of 16 or 32 columns");
  static constexpr int D = S::D, K1 = S::K1;
  static constexpr int EPT_MAX = RB / N;     // environments per tile
  static constexpr int ROWS = EPT_MAX * N;   // agent rows per tile, all in warp 0
  // B operands (rows x K, K-major, core matrices 144 bytes apart as in a_offset)
  static constexpr uint32_t X_BYTES = (RB / 8) * (K1 / 8) * kALbo;
  static constexpr uint32_t HT_BYTES = (RB / 8) * (H / 8) * kALbo;
  static constexpr uint32_t STAGE_BYTES = (ROWS * D * 4 + 15) / 16 * 16;
  static constexpr uint32_t WH_BYTES = kHeadM * H * 2;
  static constexpr int ACC_COL = 0, HEAD_COL = 32, TMEM_COLS = 64;
};

template <int N, int F, int H, int RB>
struct SmallSmem {
  using S = TcShape<N, H, false>;
  using Q = SmallShape<N, H, RB>;
  alignas(128) unsigned char weights[S::IMAGE_BYTES];
  alignas(128) unsigned char wh[Q::WH_BYTES];       // heads as a 64-row operand, rows 16.. zero
  alignas(128) unsigned char x[Q::X_BYTES];         // bf16 observations, N operand of layer 1
  alignas(128) unsigned char ht[Q::HT_BYTES];       // bf16 hidden activations, N operand of layer 2 and of the heads
  alignas(128) unsigned char stage[Q::STAGE_BYTES]; // fp32 observation block in the global layout
  alignas(16) float logit[RB * 8];                  // heads' outputs, transposed for the row threads
  alignas(8) uint32_t pub[RB * 2];                  // per row: own entity (cell, level), step count
  float uniform[RB];                                // per row: the uniform of this step's action draw
  alignas(8) uint64_t mma_bar;
  alignas(8) uint64_t load_bar;
  uint32_t tmem_base;
};

// Accumulator columns 0 .. RB-1 of this thread's lane.
template <int RB>
__device__ __forceinline__ void small_tmem_ld(uint32_t taddr, float *v) {
  if constexpr (RB == 16) {
    tmem_ld16(taddr, v);
  } else {
    uint32_t r[32];
    tmem_ld32_nowait(taddr, r);
    tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
  }
}

// Hidden unit `unit` of all rows: ReLU, bf16, into column `unit` of the hidden-activation operand.
template <int H, int RB>
__device__ __forceinline__ void small_epilogue(uint32_t acc_taddr, uint32_t ht_addr, int unit) {
  float v[RB];
  small_tmem_ld<RB>(acc_taddr, v);
#pragma unroll
  for (int n = 0; n < RB; n += 2) {
    const uint32_t p = relu_pack_bf16(__float_as_uint(v[n]), __float_as_uint(v[n + 1]));
    sts_u16(ht_addr + a_offset<H>(n, unit), static_cast<uint16_t>(p & 0xFFFFu));
    sts_u16(ht_addr + a_offset<H>(n + 1, unit), static_cast<uint16_t>(p >> 16));
  }
}

// One dense layer, weights as the M operand: accumulator[unit][row] = bias[unit] + sum_k W[unit][k] x[row][k].
template <int K, int RB, bool BIAS_TILE, int MROWS = kTileRows>
__device__ __forceinline__ void small_issue_layer(uint32_t d_tmem, uint32_t w_addr, uint32_t x_addr, uint32_t bias_addr,
                                                  uint32_t ones_addr, uint32_t bar) {
  constexpr uint32_t idesc = instr_desc(MROWS, RB);
  if (BIAS_TILE) mma_bf16(d_tmem, smem_desc(bias_addr, 128, 256), smem_desc(ones_addr, 128, 256), idesc, 0);
#pragma unroll
  for (int k = 0; k < K / 16; ++k)
    mma_bf16(d_tmem, smem_desc(w_addr + k * 256, 128, K * 16), smem_desc(x_addr + k * 2 * kALbo, kALbo, (K / 8) * kALbo),
             idesc, (BIAS_TILE || k > 0) ? 1u : 0u);
  mma_commit(bar);
}

// The thread that issues the MMAs sits in the last warp: warp 0 has the rows' serial work to do
// (stores of the previous step, the step's uniform) while a layer is being issued.
constexpr int kIssuer = kGroupThreads - 32;
constexpr int kCopier = 32;  // the thread that sends the observation block out (bulk copy)

template <int N, int F, int H, int RB, bool EVAL>
__global__ void __launch_bounds__(kGroupThreads, 1)
rollout_tc_small_kernel(RolloutArgs a, const unsigned char *__restrict__ image, int ept, int n_tiles) {
  using S = TcShape<N, H, false>;
  using Q = SmallShape<N, H, RB>;
  constexpr int D = S::D, K1 = S::K1;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  SmallSmem<N, F, H, RB> &sm = *reinterpret_cast<SmallSmem<N, F, H, RB> *>(smem_raw);
  const int row = threadIdx.x;  // hidden unit and tensor-memory lane; below RB also the agent row
  const int lane = row & 31, wg = row / 32;

  // ---- one-time set-up: barriers, tensor memory, weights -------------------------------------
  if (row == 0) {
    mbar_init(smem_u32(&sm.load_bar), 1);
    mbar_init(smem_u32(&sm.mma_bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (wg == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                 "r"(Q::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  const uint32_t w_addr = smem_u32(sm.weights), wh_addr = smem_u32(sm.wh);
  const uint32_t x_addr = smem_u32(sm.x), ht_addr = smem_u32(sm.ht), stage_addr = smem_u32(sm.stage);
  const uint32_t logit_addr = smem_u32(sm.logit), pub_addr = smem_u32(sm.pub), uni_addr = smem_u32(sm.uniform);
  for (int i = row; i < static_cast<int>(Q::X_BYTES / 16); i += kGroupThreads) sts_zero16(x_addr + 16u * i);
  for (int i = row; i < static_cast<int>(Q::HT_BYTES / 16); i += kGroupThreads) sts_zero16(ht_addr + 16u * i);
  for (int i = row; i < static_cast<int>(Q::STAGE_BYTES / 16); i += kGroupThreads) sts_zero16(stage_addr + 16u * i);
  for (int i = row; i < static_cast<int>(Q::WH_BYTES / 16); i += kGroupThreads) sts_zero16(wh_addr + 16u * i);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  bool timed_out = false;
  if (row == 0) {
    const uint32_t lbar = smem_u32(&sm.load_bar);
    mbar_expect_tx(lbar, S::IMAGE_BYTES);
    constexpr uint32_t kChunk = 16384;
    for (uint32_t off = 0; off < S::IMAGE_BYTES; off += kChunk) {
      const uint32_t n = S::IMAGE_BYTES - off < kChunk ? S::IMAGE_BYTES - off : kChunk;
      bulk_load(smem_u32(sm.weights + off), image + off, n, lbar);
    }
  }
  timed_out = !mbar_wait(smem_u32(&sm.load_bar), 0);
  timed_out = __syncthreads_or(timed_out) != 0;
  // the 16 head rows are the first two 8-row groups of the 64-row operand (same pitch)
  for (int i = row; i < static_cast<int>(S::WH_BYTES / 16); i += kGroupThreads)
    *reinterpret_cast<uint4 *>(sm.wh + 16 * i) = *reinterpret_cast<const uint4 *>(sm.weights + S::WH_OFF + 16 * i);
  fence_async_smem();
  __syncthreads();

  const uint32_t tmem_base = sm.tmem_base;
  const uint32_t lane_off = static_cast<uint32_t>(wg * 32) << 16;
  const uint32_t acc_col = tmem_base + Q::ACC_COL, head_col = tmem_base + Q::HEAD_COL;
  const uint32_t bar = smem_u32(&sm.mma_bar);
  const float *head_bias = reinterpret_cast<const float *>(sm.weights + S::BH_OFF);
  float *stage = reinterpret_cast<float *>(sm.stage);
  uint32_t phase = 0;
  bool bulk_pending = false;
  const size_t M = static_cast<size_t>(a.env.n_envs) * N;
  const int le = lane / N, ag = lane % N;  // warp 0: local environment and agent of this lane
  const int crow = le * N + ag;

  for (int tile = blockIdx.x; tile < n_tiles && !timed_out; tile += gridDim.x) {
    const int e0 = tile * ept;
    const int n_env = min(ept, a.env.n_envs - e0);
    const int n_rows = n_env * N;
    const bool active = wg == 0 && lane < Q::ROWS && le < n_env;
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
    // per-row outputs of a step wait in registers and leave while the next step's layer 1 runs
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
    auto publish = [&]() {
      if (active) {
        sts_f32(pub_addr + 8u * lane, __uint_as_float(own_entity(env, ag)));
        sts_f32(pub_addr + 8u * lane + 4u, __int_as_float(env.step));
      }
    };
    publish();
    group_sync(0);
    constexpr bool ev = EVAL;     // evaluation block: nothing of the trajectory is stored
    EvalSums sums;                // lanes with ag == 0: their environment
    for (int t = 0; t <= (ev ? a.T - 1 : a.T); ++t) {
      const bool last = !ev && (t == a.T);
      const size_t row0 = static_cast<size_t>(t) * M + static_cast<size_t>(e0) * N;
      // 1. non-zero observation entries into the zeroed operand and the zeroed fp32 block:
      //    warp 0 the level planes, warp 1 the walls, warp 2 the scalars of row = lane
      if (wg < 3 && lane < n_rows) {
        const uint32_t x_row = x_addr + a_offset<K1>(lane, 0);
        auto sink = [&](int j, float v) {
          sts_f32(stage_addr + 4u * static_cast<uint32_t>(lane * D + j), v);
          sts_u16(x_row + a_offset<K1>(0, j), bf16_bits(v));
        };
        if (wg == 0) {
          const uint32_t me = own_entity(env, ag);
          observe_levels<N, F>(env, me & 0xFF, (me >> 8) & 0xFF, sink);
        } else {
          const uint32_t me = static_cast<uint32_t>(lds_s32(pub_addr + 8u * lane));
          if (wg == 1) {
            observe_walls(me & 0xFF, (me >> 8) & 0xFF, a.env.grid, sink);
          } else {
            observe_scalars(static_cast<int>(me >> 16), lds_s32(pub_addr + 8u * lane + 4u), a.env.cap, ag, sink);
            if (S::FOLD1) {
              sts_u16(x_row + a_offset<K1>(0, D), 0x3F80);
              sts_u16(x_row + a_offset<K1>(0, D + 1), 0x3F80);
            }
          }
        }
      }
      fence_async_smem();
      tc_fence_before();
      group_sync(0);
      // 2. layer 1; meanwhile the previous step's outputs and the observation block leave
      if (wg == kIssuer / 32) {  // its other lanes wait here rather than spin beside the issuing one
        if (row == kIssuer) {
          tc_fence_after();
          small_issue_layer<K1, RB, !S::FOLD1>(acc_col, w_addr + S::W1_OFF, x_addr, w_addr + S::B1_OFF, w_addr + S::ONES_OFF,
                                               bar);
        }
        __syncwarp();
      }
      flush_outputs();
      if (!last && !ev) {
        float *obs_dst = a.buf.obs + row0 * D;
        const int count = n_rows * D;
        if (((row0 * D) & 3) == 0 && (count & 3) == 0) {
          if (row == kCopier) {
            bulk_store(obs_dst, stage_addr, static_cast<uint32_t>(count) * 4u);
            bulk_pending = true;
          }
        } else {
          for (int i = row; i < count; i += kGroupThreads) obs_dst[i] = stage[i];
        }
      }
      timed_out |= !mbar_wait(bar, phase);
      phase ^= 1;
      tc_fence_after();
      small_epilogue<H, RB>(acc_col + lane_off, ht_addr, row);
      fence_async_smem();
      tc_fence_before();
      group_sync(0);
      // 3. layer 2; meanwhile the uniform of this step's draw, and the observation operand is zeroed
      if (wg == kIssuer / 32) {  // its other lanes wait here rather than spin beside the issuing one
        if (row == kIssuer) {
          tc_fence_after();
          small_issue_layer<H, RB, true>(acc_col, w_addr + S::W2_OFF, ht_addr, w_addr + S::B2_OFF, w_addr + S::ONES_OFF, bar);
        }
        __syncwarp();
      }
      if (wg == 2 && lane < n_rows && !last)  // the uniform of row = lane, for the sampler in warp 0
        sts_f32(uni_addr + 4u * lane,
                action_uniform(a.env, a.t_global0 + static_cast<uint32_t>(t), env_id, static_cast<uint32_t>(ag)));
      for (int i = row; i < static_cast<int>(Q::X_BYTES / 16); i += kGroupThreads) sts_zero16(x_addr + 16u * i);
      if (bulk_pending) { bulk_store_wait_read(); bulk_pending = false; }  // the block may be zeroed after the next barrier
      timed_out |= !mbar_wait(bar, phase);
      phase ^= 1;
      tc_fence_after();
      small_epilogue<H, RB>(acc_col + lane_off, ht_addr, row);
      fence_async_smem();
      tc_fence_before();
      group_sync(0);
      // 4. heads: lanes 0..5 the logits, lane 6 the value, one column per row
      if (wg == kIssuer / 32) {  // its other lanes wait here rather than spin beside the issuing one
        if (row == kIssuer) {
          tc_fence_after();
          small_issue_layer<H, RB, false, kHeadM>(head_col, wh_addr, ht_addr, 0u, 0u, bar);
        }
        __syncwarp();
      }
      for (int i = row; i < static_cast<int>(Q::STAGE_BYTES / 16); i += kGroupThreads) sts_zero16(stage_addr + 16u * i);
      timed_out |= !mbar_wait(bar, phase);
      phase ^= 1;
      tc_fence_after();
      int action = 0;
      if (wg == 0) {
        float hl[RB];
        small_tmem_ld<RB>(head_col, hl);
        if (lane < 8) {
          const float b = head_bias[lane];  // the heads' biases stay fp32; entry 7 is zero
#pragma unroll
          for (int n = 0; n < RB; ++n) sts_f32(logit_addr + 4u * static_cast<uint32_t>(n * 8 + lane), hl[n] + b);
        }
        __syncwarp();
        if (active) {
          float hv[kActions + 1];
#pragma unroll
          for (int k = 0; k <= kActions; ++k) hv[k] = lds_f32(logit_addr + 4u * static_cast<uint32_t>(lane * 8 + k));
          pend = !ev; pend_step = !last; pend_row0 = row0; pend_value = hv[kActions];
          if (!last) {
            const float u = lds_f32(uni_addr + 4u * lane);
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
      // 5. transition and auto-reset, inside warp 0, which then publishes what warps 1 and 2 need
      if (wg == 0 && !last) {
        float reward;
        bool done;
        step_env_warp<N, F>(env, a.env, env_id, ag, base, active, action, reward, done);
        pend_reward = reward;
        pend_done = done;
        pend_done_idx = static_cast<size_t>(t) * a.env.n_envs + e0 + le;
        if (ev) sums.step(reward, done);
        publish();
      }
      tc_fence_before();
      if (group_any(0, timed_out)) {  // also the barrier between publishing and the next observation
        timed_out = true;
        break;
      }
      if (last) break;
    }
    flush_outputs();
    if (!timed_out && active && ag == 0) {
      store_env(env, a.state[e0 + le]);
      if (ev) { a.ev_count[e0 + le] = sums.count; a.ev_ret[e0 + le] = sums.ret; a.ev_len[e0 + le] = sums.len; }
    }
  }
  if (timed_out && row == 0) atomicExch(a.status, kStatusTimeout);
  bulk_store_wait_all();
  tc_fence_before();
  __syncthreads();
  if (wg == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(Q::TMEM_COLS) : "memory");
  }
}

template <int N, int F, int H, int RB>
cudaError_t launch_tc_small(mava_rollout *h, const RolloutArgs &args, int sms) {
  using Q = SmallShape<N, H, RB>;
  auto kern = args.eval ? rollout_tc_small_kernel<N, F, H, RB, true> : rollout_tc_small_kernel<N, F, H, RB, false>;
  const size_t smem = sizeof(SmallSmem<N, F, H, RB>);
  cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (err != cudaSuccess) return err;
  int ept = (h->cfg.n_envs + sms - 1) / sms;  // the caller made sure this fits a tile
  if (ept > Q::EPT_MAX) ept = Q::EPT_MAX;
  if (ept < 1) ept = 1;
  // A tile's observation block leaves as one bulk copy when it is a whole number of 16-byte pieces
  // (every tile then also starts on such a boundary): take the next such size if the tile has room.
  for (int e = ept; e <= Q::EPT_MAX; ++e)
    if ((e * N * Q::D) % 4 == 0) { ept = e; break; }
  const int n_tiles = (h->cfg.n_envs + ept - 1) / ept;
  kern<<<n_tiles < sms ? n_tiles : sms, kGroupThreads, smem, h->stream>>>(args, static_cast<const unsigned char *>(h->d_wtc),
                                                                         ept, n_tiles);
  h->launches += 1;
  return cudaGetLastError();
}
