// Argument structures shared by the two arithmetic paths of the update block (fp32 on the plain ALUs, bf16 on the
// tensor cores).
#pragma once
#include "common.cuh"
#include "layout.h"

namespace mava {

struct UpdNet {
  const float *W1, *b1, *W2, *b2;  // caller layout [out][in]
  const float *W1t, *W2t;          // [in][out] copies
  const float *Wa, *ba, *Wv, *bv;  // heads (nullptr when the net has none of that kind)
  int Din, H;
  size_t oW1, ob1, oW2, ob2, oWa, oba, oWv, obv;  // offsets of the gradients in the flat array
};
struct UpdRows {
  const float *x;                  // [n][Din]
  const int32_t *actions;          // [n]          (actor)
  const float *logp_old, *adv;     // [n]          (actor)
  const float *value_old, *ret;    // [n * vstride] (value), element r at r * vstride
  int vstride;
  long long n;
  // a minibatch of environments: row q of the batch is (step, env_ids[i], slot) with q = (step * n_ids + i) * per_env + slot;
  // nullptr = every environment in order (row q is row q of the arrays)
  const int32_t *env_ids;
  int n_ids, E, per_env;
};

// Row of the trajectory arrays behind row q of the batch; -1 when the environment index is out of range.
__device__ __forceinline__ long long real_row(const UpdRows &rows, long long q) {
  if (!rows.env_ids) return q;
  const long long per_step = static_cast<long long>(rows.n_ids) * rows.per_env;
  const long long t = q / per_step, rem = q - t * per_step;
  const int i = static_cast<int>(rem / rows.per_env), slot = static_cast<int>(rem - static_cast<long long>(i) * rows.per_env);
  const int e = rows.env_ids[i];
  if (e < 0 || e >= rows.E) return -1;
  return (t * rows.E + e) * rows.per_env + slot;
}

struct UpdHyper { float clip_eps, ent_coef, vf_coef; };

// Tensor-core path (update_tc.cu): shared-torso nets with H <= 128 and D <= 80.
bool ppo_tc_supported(const mava_config_t &cfg, int D);
size_t ppo_tc_image_bytes();
// Enqueues the weight-image kernel and the loss/gradient kernel; `partial` holds `slices` slices of n_params floats
// (one per CTA, every parameter written once per slice), `term_partial` 8 x 3 doubles per slice.
cudaError_t launch_ppo_net_tc(mava_rollout *h, const float *params_dev, const ParamLayout &L, const UpdRows &rows, const UpdHyper &hp,
                              const double *adv_stats, void *image, float *partial, size_t n_params, double *term_partial, int slices);


// Tensor-core path for H = 256 (update_tc256.cu): a net with hidden width 256 whose first layer takes `slabs` observation
// slabs of width 64 < D <= 96 side by side (1: the actor / shared-torso net; n_agents: the centralised critic), a chunk
// of `chunk_tiles` 128-row tiles at a time through `staging` (ppo_tc256_staging_bytes bytes).  Offsets are those of the
// net's layers in the flat parameter array.  Adds into the slices of `partial` and into `term_partial` (both zeroed by
// the caller); needs slices >= 1 + slabs.
struct Tc256Net {
  size_t W1, b1, W2, b2, Wa, ba, Wv, bv;
  int slabs;
  bool has_actor, has_value;
};
bool ppo_tc256_supported(const mava_config_t &cfg, int D);
size_t ppo_tc256_image_bytes(int slabs);
size_t ppo_tc256_staging_bytes(int chunk_tiles, int slabs);
cudaError_t launch_ppo_net_tc256(mava_rollout *h, const float *params_dev, const Tc256Net &net, const UpdRows &rows, const UpdHyper &hp,
                                 const double *adv_stats, void *image, void *staging, int chunk_tiles, float *partial, size_t n_params,
                                 double *term_partial, int slices);

}  // namespace mava
