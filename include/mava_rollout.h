/*
 * mava_rollout.h -- C ABI of the fused multi-agent rollout + GAE library (CUDA, sm_100a).
 *
 * The library runs, entirely on one GPU, the experience-collection stage of the Anakin
 * training loop of the Mava technical report (Section 2, "Strong baseline algorithms and
 * training architectures", and Figure 2: every update function steps its own batch of
 * environment copies), followed by advantage estimation for the multi-agent PPO systems the
 * report names (IPPO with per-agent critics, MAPPO with a centralised critic).
 *
 * E level-based-foraging gridworlds (the report's LBF tasks, Section 4) with N agents
 * each are stepped T times.  One step, per environment:
 *     observe -> actor/critic MLP forward -> categorical sample (Philox4x32-10,
 *     inverse CDF) -> environment transition -> auto-reset when the episode ended.
 *
 * General rules
 *   - Every function returns MAVA_OK (0) or a negative MAVA_ERR_* code; nothing throws,
 *     aborts or exits.  mava_strerror() names a code.
 *   - "device pointer" = memory of the CUDA device that was current at create time;
 *     "host pointer" = ordinary (preferably pinned) host memory.
 *   - Work is enqueued on the stream given at create time and the call returns without
 *     waiting, unless stated otherwise.  Problems found by a kernel (a bounded wait that
 *     ran out) are recorded in a device status word that mava_rollout_status() reads.
 *   - The caller owns the trajectory buffers and the parameters; the library owns only
 *     the handle and its small internal device state (environment states, re-laid-out
 *     weights, status word), allocated at create and freed at destroy.
 *   - The library has no CPU fallback: without a CUDA device create fails.
 */
#ifndef MAVA_ROLLOUT_H
#define MAVA_ROLLOUT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MAVA_OK 0
#define MAVA_ERR_INVALID_ARG (-1)    /* null pointer, non-positive size, value out of range      */
#define MAVA_ERR_UNSUPPORTED (-2)    /* shape outside the compiled table, or not an sm_100 GPU   */
#define MAVA_ERR_CUDA (-3)           /* a CUDA runtime call failed                               */
#define MAVA_ERR_DEVICE_TIMEOUT (-4) /* a bounded device-side wait gave up (see status)          */
#define MAVA_ERR_CAPACITY (-5)       /* T larger than max_T, or a size beyond a stated maximum   */

#define MAVA_N_ACTIONS 6 /* 0 noop, 1 up (r-1), 2 down (r+1), 3 left (c-1), 4 right (c+1), 5 load */

#define MAVA_ENV_FORAGING 0  /* level-based foraging (the rules in the general comment above)           */
#define MAVA_ENV_WAREHOUSE 1 /* warehouse: robots carry requested shelves to the delivery row             */
#define MAVA_ENV_WAREHOUSE_CONFLICTS_END 2 /* the same, and a robot conflict ends the episode             */

#define MAVA_NET_SHARED_TORSO 0 /* one torso, a 6-logit actor head and a value head (IPPO-style)   */
#define MAVA_NET_CENTRAL_CRITIC 1 /* actor net per agent + critic on the joint observation (MAPPO) */

#define MAVA_NET_RECURRENT 2 /* recurrent policy: dense ReLU embedding, one gated recurrent unit of width H that
                                carries a hidden vector per agent, actor and value heads on the new hidden vector */

#define MAVA_PRECISION_FP32 0 /* fp32 SIMT arithmetic (validation path)                            */
#define MAVA_PRECISION_BF16 1 /* bf16 operands, fp32 accumulation on the tcgen05 tensor cores      */

#define MAVA_FLAG_WRITE_LOGITS 1 /* also write the six logits of every row to buffers.logits       */
#define MAVA_FLAG_HIDDEN_IN_TMEM 2 /* bf16 path, H = 64: keep hidden activations in tensor memory (the layout the 128-row
                                      kernel always uses from H = 128 on); at H = 128 the flag only selects the 128-row
                                      kernel like MAVA_FLAG_WIDE_TILES; results are identical */
#define MAVA_FLAG_WIDE_TILES 4 /* bf16 path: always use 128-row tiles, also for batches small
                                  enough for the few-rows form of the kernel; results are identical */

#define MAVA_FLAG_UPDATE_FP32 8 /* bf16 handle: the update block (mava_ppo_grad*) still computes in fp32 on the
                                  plain ALUs instead of taking the tensor-core kernels */

typedef struct mava_rollout mava_rollout_t; /* opaque, owned by the library */

/* Plain data, copied at create.  The observation width is D = 3*(2*view_radius+1)^2 + 2 + n_agents. */
typedef struct {
  int32_t grid;            /* G: playable area is G x G cells; everything outside is wall         */
  int32_t n_agents;        /* N agents per environment                                            */
  int32_t n_food;          /* F food items per environment                                        */
  int32_t max_agent_level; /* agent levels are uniform in 1..max_agent_level (at most 3)          */
  int32_t view_radius;     /* egocentric window radius; only 2 is compiled                        */
  int32_t episode_cap;     /* an episode ends when its step count reaches this                    */
  int32_t n_envs;          /* E                                                                   */
  int32_t max_T;           /* capacity, in steps, of the caller's trajectory buffers              */
  int32_t hidden;          /* H, width of both hidden layers                                      */
  int32_t net_kind;        /* MAVA_NET_*                                                          */
  int32_t precision;       /* MAVA_PRECISION_*                                                    */
  int32_t flags;           /* MAVA_FLAG_* bits                                                    */
  int32_t first_env;       /* global index of this handle's environment 0 (keys Philox), so that
                              shards of one large batch reproduce the unsharded run; usually 0    */
  int32_t env_kind;        /* MAVA_ENV_*: the workload family (0 = level-based foraging)          */
  uint64_t seed;           /* keys every Philox stream                                            */
} mava_config_t;

/* Device pointers to caller-owned, time-major trajectory buffers (M = E*N agent rows per step).
 * adv/ret may be NULL if mava_gae is never called; logits may be NULL unless
 * MAVA_FLAG_WRITE_LOGITS is set.  All must stay valid until destroy.  obs must be 16-byte
 * aligned. */
typedef struct {
  float *obs;       /* [max_T][E][N][D]  observation each agent acted on                       */
  int32_t *actions; /* [max_T][E][N]     action taken                                          */
  float *logp;      /* [max_T][E][N]     log-probability of that action                        */
  float *values;    /* [max_T+1][E][N]   critic value of the row; row T = bootstrap            */
  float *rewards;   /* [max_T][E][N]     shared reward, replicated over the env's agents       */
  uint8_t *dones;   /* [max_T][E]        1 when the step ended the episode                     */
  float *adv;       /* [max_T][E][N]     GAE advantages                                        */
  float *ret;       /* [max_T][E][N]     returns = advantages + values                         */
  float *logits;    /* [max_T][E][N][6]  optional                                              */
} mava_buffers_t;

/* The same arrays in host memory, for mava_rollout_collect_host (any pointer may be NULL to
 * skip that array). */
typedef mava_buffers_t mava_host_buffers_t;

/* Number of floats in the flat parameter array.  Layout: dense layers as weight[out][in]
 * (y = x W^T + b) followed by bias[out], in this order
 *   MAVA_NET_SHARED_TORSO:   W1[H][D] b1  W2[H][H] b2  Wa[6][H] ba  Wv[1][H] bv
 *   MAVA_NET_CENTRAL_CRITIC: W1[H][D] b1  W2[H][H] b2  Wa[6][H] ba  (actor, per agent)
 *                            C1[H][N*D] c1  C2[H][H] c2  Cv[1][H] cv (critic; its input is the
 *                            observations of agents 0..N-1 concatenated)
 *   MAVA_NET_RECURRENT:      W1[H][D] b1  Wih[3H][H] bih[3H]  Whh[3H][H] bhh[3H]  Wa[6][H] ba  Wv[1][H] bv
 * ReLU follows both hidden layers; heads are linear.  Recurrent policy (Section 2 names recurrent versions of every
 * system and Section 4 reports them on LBF; no cell or size is given, so this is the library's reading): e = relu(W1 x +
 * b1); gated recurrent unit of Cho et al. (2014) with the gate blocks r, z, n stacked in that order,
 *   r = sigma(Wir e + bir + Whr h + bhr);  z = sigma(Wiz e + biz + Whz h + bhz);
 *   n = tanh(Win e + bin + r * (Whn h + bhn));  h' = (1 - z) * n + z * h;
 * heads on h'.  The hidden vector of every agent is zero at create/reset and restarts from zero whenever its
 * environment's episode ends; the handle carries it from one run to the next.  The bootstrap row values[T] comes from
 * one more cell update on the observation after the last step, which is not kept.  Returns 0 for an invalid config. */
size_t mava_params_count(const mava_config_t *cfg);

/* Validates cfg, allocates the handle and its device state on the current device, places every
 * environment at the start of episode 0 (positions and levels from Philox keyed by
 * (seed, env, episode)) and stores the handle in *out.  `cuda_stream` is a cudaStream_t (NULL =
 * default stream).  Synchronous.  Errors: INVALID_ARG, UNSUPPORTED, CUDA. */
int mava_rollout_create(const mava_config_t *cfg, const mava_buffers_t *buffers, void *cuda_stream,
                        mava_rollout_t **out);

/* The fused rollout (the per-update experience collection of Figure 2).  Continues from the handle's environment states for T steps (1 <= T <= max_T),
 * writing rows 0..T-1 of obs, actions, logp, values, rewards, dones (and logits when flagged) and
 * the bootstrap row values[T].  params_dev: device pointer to mava_params_count floats, read
 * during the call's kernels (must stay valid until they finish).  With the central critic the one
 * value of an environment is written to all its N slots.  Asynchronous.
 * Errors: INVALID_ARG, CAPACITY, CUDA. */
int mava_rollout_run(mava_rollout_t *h, const float *params_dev, int32_t T);

/* Same, but every action is taken from actions_dev ([T][E][N] int32, device pointer, values 0..5)
 * instead of being sampled ("teacher forcing"); the given actions are copied to buffers.actions
 * and logp is that of the forced action. */
int mava_rollout_run_forced(mava_rollout_t *h, const float *params_dev, int32_t T,
                            const int32_t *actions_dev);

/* Evaluation block (Section 2, "Multi-device training with easy checkpointing and logging":
 * training is interleaved with blocks that run the current policy to report how it does).  The
 * same loop as the rollout for T >= 1 steps (not limited by max_T), continuing from the handle's
 * environment states and step counter and advancing both, but nothing of the trajectory is stored
 * and the caller's buffers are not touched.  greedy != 0: every action is the arg max of its six
 * logits, the lowest index on a tie; greedy == 0: the rollout's Philox draw.  Outputs, device
 * pointers to n_envs elements each, written by the call's kernels, over the episodes that END
 * inside the block: ep_count how many, ret_sum the sum of their returns (an episode's return is
 * the sum of its shared step rewards received inside the block; fp32 sums in step order), len_sum
 * the sum of their lengths in steps inside the block.  An episode still running at the end of the
 * block is not counted.  actions_dev: NULL, or [T][E][N] int32 that receives the actions taken.
 * The centralised critic is not evaluated.  Asynchronous.  Errors: INVALID_ARG, CUDA. */
int mava_rollout_evaluate(mava_rollout_t *h, const float *params_dev, int32_t T, int32_t greedy,
                          int32_t *ep_count_dev, float *ret_sum_dev, int32_t *len_sum_dev,
                          int32_t *actions_dev);

/* Generalised advantage estimation over the rows of the last run (multi-agent PPO, Section 2):
 *   delta_t = r_t + gamma V_{t+1} (1-d_t) - V_t;  A_t = delta_t + gamma lambda (1-d_t) A_{t+1},
 *   A_T = 0;  Ret_t = A_t + V_t.
 * Reads values, rewards, dones; writes adv and ret.  Handles runs of up to MAVA_GAE_MAX_T steps.  Asynchronous.
 * Errors: INVALID_ARG (no run yet, adv/ret NULL, gamma or lambda outside [0, 1]), CAPACITY (the last run
 * was longer than MAVA_GAE_MAX_T steps), CUDA. */
#define MAVA_GAE_MAX_T 1024
int mava_gae(mava_rollout_t *h, float gamma, float lambda);

/* Update block (Section 2: each update function minimises the multi-agent PPO loss on the rolled-out experience;
 * the report prints no formula, so the clipped-surrogate objective of Schulman et al. 2017 is taken, see below).
 * Coefficients of the loss and of the optimiser; mava_ppo_defaults fills in 0.2, 0.01, 0.5, 2.5e-4, 0.9, 0.999,
 * 1e-5, 0.5. */
typedef struct {
  float clip_eps, ent_coef, vf_coef;          /* loss */
  float lr, beta1, beta2, adam_eps;           /* Adam */
  float max_grad_norm;                        /* global 2-norm the gradient is scaled down to */
} mava_ppo_hyper_t;
void mava_ppo_defaults(mava_ppo_hyper_t *hp);

/* Loss and gradient of one minibatch made of ALL rows of the last run (T steps; mava_gae must have run), under
 * `params_dev` (same layout as for run):
 *   rho = exp(logp_new(a) - logp);  Ahat = (adv - mean adv) / (std adv + 1e-8)   (population std over the rows)
 *   L = -mean min(rho Ahat, clip(rho, 1 - eps, 1 + eps) Ahat) - ent_coef * mean H
 *       + vf_coef * 0.5 * mean max((V - ret)^2, (values + clip(V - values, -eps, eps) - ret)^2)
 * With the centralised critic a value row is an environment-step (slot 0 of `values` and `ret`, its input the
 * agents' observations concatenated).  Reads obs, actions, logp, values, adv, ret of the caller's buffers; writes
 * grad_dev [mava_params_count] (dL/dparams, parameter order) and, if not NULL, terms_dev [4] = L, actor term,
 * mean entropy, value term (device pointers).
 * Arithmetic: an fp32 handle computes in fp32 on the plain ALUs.  A bf16 handle takes tensor-core kernels (bf16
 * operands, fp32 accumulation; the derivatives with respect to the hidden pre-activations are rounded to bf16 before
 * they enter a product) for the shared-torso shapes with H <= 128 and for H = 256 (with the centralised critic: both
 * nets), unless MAVA_FLAG_UPDATE_FP32 is set.  The rollout of a bf16 handle
 * stored logp and values from bf16 arithmetic: re-evaluated at unchanged parameters by the tensor-core kernels (same
 * operand rounding) the ratio rho is 1 to about 1e-3; re-evaluated in fp32 (the flag) the rollout's rounding shows as
 * a policy change of up to a few 1e-2 in rho and in V - values, which the clips then see.
 * The library allocates its scratch on the first call and keeps it until destroy: one gradient slice of params_count
 * floats per resident CTA (up to three per SM), and for H = 256 on the tensor cores a staging buffer of up to 1.5 GB.
 * The recurrent policy has no update block (MAVA_ERR_UNSUPPORTED).  Asynchronous.
 * Errors: INVALID_ARG (NULL pointers, no run yet, adv/ret NULL), UNSUPPORTED, CUDA. */
int mava_ppo_grad(mava_rollout_t *h, const float *params_dev, const mava_ppo_hyper_t *hp, float *grad_dev, float *terms_dev);

/* The same over a minibatch of environments: the rows of the n_ids environments env_ids_dev[0..n_ids) (device
 * pointer, local indices 0..n_envs-1, any order; a repeated index counts twice) at every step of the last run; the
 * advantages are normalised over that minibatch.  A permutation of all environments cut into pieces gives the
 * shuffled minibatches of a PPO epoch.  An index outside 0..n_envs-1 makes the kernel skip that environment's rows
 * and mava_rollout_status answer MAVA_ERR_INVALID_ARG.  Errors: as mava_ppo_grad, and INVALID_ARG for n_ids < 1. */
int mava_ppo_grad_envs(mava_rollout_t *h, const float *params_dev, const mava_ppo_hyper_t *hp, const int32_t *env_ids_dev,
                       int32_t n_ids, float *grad_dev, float *terms_dev);

/* One Adam step in place (Kingma & Ba 2015, bias-corrected; `step` counts from 1) after the gradient has been
 * scaled to a global 2-norm of at most max_grad_norm:  m = b1 m + (1 - b1) g;  v = b2 v + (1 - b2) g^2;
 * params -= lr * (m / (1 - b1^step)) / (sqrt(v / (1 - b2^step)) + adam_eps).  All arrays are device pointers of
 * mava_params_count floats; m and v start at zero and belong to the caller.  Asynchronous.
 * Errors: INVALID_ARG (NULL pointers, step < 1), CUDA. */
int mava_adam_step(mava_rollout_t *h, float *params_dev, const float *grad_dev, float *m_dev, float *v_dev, int32_t step,
                   const mava_ppo_hyper_t *hp);

/* The update loop of one training iteration behind one call (Section 2, Figure 2: each update function turns its
 * rolled-out experience into new parameters): `epochs` passes over the last run's rows, each pass cut into
 * `minibatches` minibatches of environments, every minibatch one mava_ppo_grad_envs followed by one mava_adam_step
 * (step numbers first_step, first_step + 1, ...).  The shuffling is the caller's: perm_dev is [epochs][n_envs] int32
 * (device pointer), row e a permutation of 0..n_envs-1 (any list of valid indices works; it is not checked beyond the
 * range check of mava_ppo_grad_envs); minibatch k of pass e is the slice [k * n_envs / minibatches, (k + 1) * n_envs /
 * minibatches) of that row.  params_dev, m_dev, v_dev are updated in place; grad_dev is workspace of
 * mava_params_count floats; terms_dev, if not NULL, receives [epochs * minibatches][4] loss terms in the order the
 * minibatches were taken.  Asynchronous: everything is enqueued on the handle's stream, nothing is copied to the host.
 * Errors: as mava_ppo_grad_envs and mava_adam_step; INVALID_ARG for epochs < 1, minibatches < 1 or > n_envs. */
int mava_ppo_update(mava_rollout_t *h, float *params_dev, float *m_dev, float *v_dev, float *grad_dev, const mava_ppo_hyper_t *hp,
                    int32_t epochs, int32_t minibatches, const int32_t *perm_dev, int32_t first_step, float *terms_dev);

/* Back to episode 0 and global step 0 under a new seed.  Asynchronous. */
int mava_rollout_reset(mava_rollout_t *h, uint64_t seed);

/* Waits for the stream, then returns MAVA_OK, MAVA_ERR_DEVICE_TIMEOUT if a kernel's bounded wait
 * gave up since the last call, MAVA_ERR_INVALID_ARG if a kernel met an environment index out of range
 * (the status word is cleared either way), or MAVA_ERR_CUDA. */
int mava_rollout_status(mava_rollout_t *h);

/* Environment states as int32 records of mava_state_record_len(cfg) words per environment:
 * N x (row, col, level), F x (row, col, level; level 0 = collected), step, episode,
 * total food level at reset.  Host pointers; both calls wait for the stream.  set validates
 * ranges (INVALID_ARG) and leaves the global step counter unchanged. */
int32_t mava_state_record_len(const mava_config_t *cfg);
int mava_rollout_get_state(mava_rollout_t *h, int32_t *records_host);
int mava_rollout_set_state(mava_rollout_t *h, const int32_t *records_host);

/* Recurrent policy: copies the hidden vectors the next run will start from, [E][N][H] fp32, to host memory (waits
 * for the stream).  Errors: INVALID_ARG (also when the handle's net is not recurrent), CUDA. */
int mava_rollout_get_hidden(mava_rollout_t *h, float *hidden_host);

/* End-to-end convenience with HOST buffers: copies params_host to the device, runs T steps and
 * GAE, copies every non-NULL array of `out` back to the host (rows 0..T-1; T+1 rows of values)
 * and waits.  The caller's device buffers given at create are used as staging.  Synchronous.
 * Errors: as run and gae. */
int mava_rollout_collect_host(mava_rollout_t *h, const float *params_host, int32_t T, float gamma,
                              float lambda, const mava_host_buffers_t *out);

/* Allocation-free rollout (the paper has no counterpart; it exists for callers that cannot
 * allocate).  Some users of this library must not call cudaMalloc/cudaFree while they run: a
 * process that handed all device memory to its own pool, a serving or control loop in which the
 * implicit device-wide synchronisation of an allocation is not acceptable, or code that runs after
 * its start-up phase under a "no further allocations" rule.  This entry point does what
 * create + run do for a fresh handle -- every environment starts episode 0 at global step 0 under
 * cfg->seed, then T steps are rolled out into the caller's buffers -- but it creates no handle
 * and calls no allocating routine: the library's scratch (status word, environment states,
 * re-laid-out weights) lives in one static device array of MAVA_STATIC_SCRATCH_BYTES that every
 * GPU loading the library holds until the process exits.
 *   - The scratch of a shape is 256 bytes + 60 bytes per environment + the re-laid-out weights, each part
 *     rounded up to 256 bytes.  The weights depend on the shape and the precision: bf16 images take 18 KB
 *     (H = 64), 70 KB (H = 128) or 205 KB (H = 256, about 13 000 environments fit beside them); the fp32 path
 *     keeps 4 bytes per parameter (24 KB ... 350 KB for the shared-torso shapes, 930 KB with the centralised
 *     critic, which leaves room for about 1 600 environments).  A shape whose scratch is larger than the
 *     array is refused with MAVA_ERR_CAPACITY, and so is T > cfg->max_T.  The bf16 path with the centralised
 *     critic needs far more scratch than the array (critic weight images and an observation block) and is
 *     refused with MAVA_ERR_UNSUPPORTED: use the fp32 path or a handle.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress);
 *     make that first call before any stream capture.
 *   - All calls share the array and it keeps the previous call's contents; the call clears what
 *     must start at zero.  Two calls that overlap on the GPU (different streams or threads) race:
 *     serialise them.  It does not touch handles made by mava_rollout_create.
 *   - cfg, buffers, params_dev and T mean what they mean for create and run.  GAE is not included and
 *     cannot be reached from here: mava_gae works on a handle made by mava_rollout_create (which
 *     allocates).  The call waits for the stream and returns MAVA_OK, MAVA_ERR_DEVICE_TIMEOUT, or the
 *     errors of create/run. */
#define MAVA_STATIC_SCRATCH_BYTES (1u << 20)
int mava_rollout_run_static(const mava_config_t *cfg, const mava_buffers_t *buffers, const float *params_dev,
                            int32_t T, void *cuda_stream);

/* Self-test hook of the failure-detection path (no counterpart in the report).  Every wait of a kernel on an
 * mbarrier is bounded; when one runs out the kernel records it in the status word, lets the copies it still has
 * in flight land, frees its tensor memory and returns, and mava_rollout_status answers MAVA_ERR_DEVICE_TIMEOUT.
 * This call arms the NEXT launch of `which` (MAVA_EXPIRE_GAE: the copy-engine GAE kernel; MAVA_EXPIRE_ROLLOUT:
 * the 128-row tensor-core rollout kernel) so that one thread block makes one extra wait, with a limit of a few
 * thousand polls, on a barrier phase that nothing will complete, at a point where none of its copies or MMAs is
 * outstanding.  That block gives up exactly as after a real time-out; its outputs (and, for the rollout, the
 * environment states of its tile) are then incomplete, so the caller resets the handle afterwards.  One launch
 * only; a launch that takes another kernel (a shape the armed kernel does not serve) leaves the request armed.
 * Errors: INVALID_ARG. */
#define MAVA_EXPIRE_GAE 1
#define MAVA_EXPIRE_ROLLOUT 2
int mava_debug_expire_next_wait(mava_rollout_t *h, int32_t which);

/* Number of kernels this handle has launched so far (for launch accounting). */
int64_t mava_rollout_launch_count(const mava_rollout_t *h);

/* Frees the handle and its device state after waiting for the stream.  NULL is allowed. */
void mava_rollout_destroy(mava_rollout_t *h);

const char *mava_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* MAVA_ROLLOUT_H */
