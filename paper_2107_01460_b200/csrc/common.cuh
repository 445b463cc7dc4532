// Internal declarations shared by the translation units of libmava_rollout.so.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "mava_rollout.h"

namespace mava {

constexpr int kCollectChunks = 4;  // pieces (in time) a host-collected rollout is cut into
constexpr int kMaxAgents = 8;
constexpr int kMaxFood = 8;
constexpr int kActions = MAVA_N_ACTIONS;
constexpr int kViewRadius = 2;
constexpr int kWindow = 2 * kViewRadius + 1;       // 5
constexpr int kPlane = kWindow * kWindow;          // 25
constexpr int kObsFixed = 3 * kPlane + 2;          // 77: three planes, own level, step/cap

constexpr uint32_t kDomainReset = 0x52534554u;     // key tweak of the placement stream
constexpr uint32_t kDomainAction = 0x41435431u;    // key tweak of the action-uniform stream

// Device status word values (0 = fine).
constexpr int kStatusTimeout = 1;
constexpr int kStatusBadIndex = 2;  // an environment index of a minibatch was out of range (its rows were skipped)

// Compact per-environment state.  Coordinates and levels fit a byte (G <= 64, levels <= 31).
struct __align__(4) EnvRec {
  uint8_t ar[kMaxAgents], ac[kMaxAgents], al[kMaxAgents];
  uint8_t fr[kMaxFood], fc[kMaxFood], fl[kMaxFood];  // fl == 0: collected
  int32_t step, episode, total;
};
static_assert(sizeof(EnvRec) == 60, "EnvRec layout");

// Runtime scalars every kernel needs.
struct EnvParams {
  int32_t grid, max_level, cap, n_envs;
  int32_t first_env;        // global index of local environment 0 (Philox is keyed on global indices)
  uint32_t key_lo, key_hi;  // seed halves (domain tweak applied on use)
  int32_t env_kind;         // 0: foraging; 1: warehouse; 2: warehouse whose episode ends on a robot conflict
};

// Everything a rollout launch needs.
struct RolloutArgs {
  EnvParams env;
  mava_buffers_t buf;
  EnvRec *state;
  const int32_t *forced;  // [T][E][N] or nullptr
  int32_t T;
  uint32_t t_global0;
  int32_t write_logits;
  int *status;
  float *obs_last;  // bf16 path with a centralised critic: where the observation after the last step goes
  // Evaluation block: no trajectory is stored; per environment the episodes ending inside the block
  // are counted and their returns and lengths summed.
  int32_t eval;         // 0: rollout, 1: evaluation block
  int32_t greedy;       // evaluation: arg max of the logits (lowest index on a tie) instead of the draw
  int32_t *ev_count;    // [E]
  float *ev_ret;        // [E]
  int32_t *ev_len;      // [E]
  int32_t *ev_actions;  // [T][E][N] or nullptr
  // Self-test of the give-up path: block 0's first thread group makes one extra, short, bounded wait that nothing
  // completes (after step 1's heads, when none of its MMAs or copies is outstanding) and treats it as a time-out.
  int32_t debug_expire;
};

// Episode bookkeeping of one environment inside an evaluation block (all in step order, fp32 sums).
struct EvalSums {
  float running = 0.0f, ret = 0.0f;  // return of the episode in progress; sum over the finished ones
  int32_t length = 0, len = 0, count = 0;
  __device__ __forceinline__ void step(float reward, bool done) {
    running += reward;
    length += 1;
    if (done) {
      count += 1; ret += running; len += length;
      running = 0.0f; length = 0;
    }
  }
};

// Index of the largest of the six logits, the lowest index on a tie.
__device__ __forceinline__ int greedy_action(const float *l) {
  int best = 0;
  float top = l[0];
#pragma unroll
  for (int k = 1; k < kActions; ++k)
    if (l[k] > top) { top = l[k]; best = k; }
  return best;
}

// Re-laid-out fp32 weights of the SIMT path: every dense layer transposed to [in][out].
struct SimtWeights {
  const float *W1t, *b1, *W2t, *b2, *Wa, *ba, *Wv, *bv;  // Wa [6][H], Wv [H] stay row-major
  const float *C1t, *c1, *C2t, *c2, *Cv, *cv;            // central critic (or nullptr)
};

}  // namespace mava

struct mava_rollout {
  mava_config_t cfg;
  mava_buffers_t buf;
  cudaStream_t stream;
  int device;
  int D;            // observation width
  int variant;      // index in the compiled shape table
  mava::EnvRec *d_state;
  int *d_status;
  float *d_wsimt;   // transposed fp32 weights (SIMT path)
  void *d_wtc;      // bf16 weights in tensor-core layout (bf16 path)
  float *d_params_stage;  // device copy of host params (collect_host)
  void *d_critic;      // centralised critic on the bf16 path: weight images
  float *d_obs_last;   //   and the observations after the last step [E][N][D]
  void *d_upd;         // scratch of the update block (made on its first call)
  size_t upd_bytes;
  float *d_hidden;     // recurrent policy: the agents' hidden vectors [E][N][H]
  void *d_upd_stage;   // staging buffer of the H = 256 tensor-core update (made on its first call)
  size_t upd_stage_bytes;
  uint32_t t_global;
  int32_t last_T;
  int64_t launches;
  int32_t expire_next;  // MAVA_EXPIRE_* bits armed by mava_debug_expire_next_wait
  // collect_host: a second stream carries the device-to-host copies of the steps already rolled
  // out while the rest of the rollout runs (created on first use)
  cudaStream_t copy_stream;
  cudaEvent_t chunk_done[mava::kCollectChunks + 1];
  bool copy_ready;
};

namespace mava {

// Shape table: the (N, F, H, net_kind) combinations kernels are compiled for.
int find_variant(const mava_config_t &cfg);  // -1 if not compiled

// Launchers (each returns a cudaError_t; all asynchronous on h->stream).
cudaError_t launch_env_init(mava_rollout *h);
cudaError_t launch_prep_simt(mava_rollout *h, const float *params_dev);
cudaError_t launch_rollout_simt(mava_rollout *h, const RolloutArgs &args);
cudaError_t launch_gae(mava_rollout *h, float gamma, float lambda);
size_t simt_weight_floats(const mava_config_t &cfg, int D);

// bf16 tensor-core path.
size_t tc_weight_bytes(const mava_config_t &cfg, int D);
cudaError_t launch_prep_tc(mava_rollout *h, const float *params_dev);
cudaError_t launch_rollout_tc(mava_rollout *h, const RolloutArgs &args);
bool tc_supported(const mava_config_t &cfg);
bool tc_rollout_is_wide(const mava_rollout *h);  // the next bf16 rollout launch takes the 128-row kernel (not the few-rows form)
size_t critic_weight_bytes(const mava_config_t &cfg);
cudaError_t launch_critic_tc(mava_rollout *h, const float *params_dev, int32_t T);

// Recurrent policy (rollout_rec.cu: fp32 SIMT; rollout_rec_tc.cu: bf16 tensor cores).
cudaError_t launch_rollout_rec_simt(mava_rollout *h, const float *params_dev, const RolloutArgs &args);
cudaError_t launch_rollout_rec_tc(mava_rollout *h, const float *params_dev, const RolloutArgs &args);
size_t rec_tc_weight_bytes(const mava_config_t &cfg);

// Update block (fp32).
cudaError_t launch_ppo_grad(mava_rollout *h, const float *params_dev, const mava_ppo_hyper_t &hp, float *grad_dev, float *terms_dev,
                            const int32_t *env_ids_dev, int32_t n_ids);
cudaError_t launch_adam_step(mava_rollout *h, float *params_dev, const float *grad_dev, float *m_dev, float *v_dev, int32_t step,
                             const mava_ppo_hyper_t &hp);

}  // namespace mava
