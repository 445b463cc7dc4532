/*
 * CPU oracle for the batched multi-agent rollout + GAE path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, obviously-correct
 * restatement of what the rollout computes: the foraging gridworld
 * (reset, observation, transition, reward, done), the shared actor-critic MLP,
 * the Philox4x32-10 inverse-CDF categorical sampler, generalised advantage
 * estimation, the evaluation block (greedy or sampled episodes, returns) and
 * the recurrent (gated-recurrent-unit) policy.  It shares no code with the CUDA library and is used only by the
 * tests, by the smoke check and by the benchmark's CPU-baseline leg.
 *
 * The technical report this follows describes the loop only in words
 * (Section 2, "Strong baseline algorithms and training architectures", and the
 * caption of Figure 2: every update function rolls out experience from N
 * vectorised environment copies and hands it to a loss).  The concrete rules
 * are those of the synthetic level-based foraging workload that stands in for
 * the paper's LBF tasks (Section 4, "Level-Based Foraging"); each function
 * below states the rule it implements.
 *
 * Floating point: the MLP, softmax and GAE accumulate in double.  Quantities
 * the method fixes in single precision (observation entries, the reward
 * quotient, the Philox uniform) are computed with one IEEE binary32 operation.
 *
 * Every function here has at least one independent pin in tests/ (known-answer
 * vectors, hand-worked transitions, closed forms, brute force, library
 * referees); none is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_MAX_AGENTS 8
#define ORC_MAX_FOOD 8
#define ORC_N_ACTIONS 6

#define ORC_DOMAIN_RESET 0x52534554u  /* key tweak for placement draws  */
#define ORC_DOMAIN_ACTION 0x41435431u /* key tweak for action uniforms  */
#define ORC_DOMAIN_REQUEST 0x52455153u /* key tweak for the warehouse's new requests */

typedef struct {
  int32_t grid;            /* G: playable cells are rows/cols 0..G-1            */
  int32_t n_agents;        /* N                                                 */
  int32_t n_food;          /* F                                                 */
  int32_t max_agent_level; /* agent level uniform in 1..max_agent_level         */
  int32_t view_radius;     /* R: egocentric window is (2R+1) x (2R+1)           */
  int32_t episode_cap;     /* episode ends when step reaches this               */
  int32_t hidden;          /* H: width of both hidden layers                    */
  int32_t net_kind;        /* 0: shared torso + actor/value heads
                              1: actor net + centralised critic on joint obs
                              2: recurrent policy                               */
  int32_t env_kind;        /* 0: level-based foraging; 1: warehouse;
                              2: warehouse whose episode ends on a robot conflict */
} orc_config_t;

typedef struct {
  int32_t agent_r[ORC_MAX_AGENTS], agent_c[ORC_MAX_AGENTS], agent_level[ORC_MAX_AGENTS];
  int32_t food_r[ORC_MAX_FOOD], food_c[ORC_MAX_FOOD], food_level[ORC_MAX_FOOD]; /* 0 = gone */
  int32_t step;             /* steps already taken in this episode */
  int32_t episode;          /* episode index of this env           */
  int32_t total_food_level; /* sum of food levels at reset         */
} orc_env_state_t;

int32_t orc_obs_dim(const orc_config_t *cfg) {
  int32_t w = 2 * cfg->view_radius + 1;
  return 3 * w * w + 2 + cfg->n_agents;
}

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as    */
/* easy as 1, 2, 3", SC'11): ten rounds; each round multiplies counter words  */
/* 0 and 2 by two fixed constants, swaps/xors the halves with the key, and    */
/* the key is bumped by two Weyl constants between rounds.                    */
/* ------------------------------------------------------------------------- */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    uint32_t n0 = hi1 ^ c1 ^ k0;
    uint32_t n1 = lo1;
    uint32_t n2 = hi0 ^ c3 ^ k1;
    uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Integer in [0, n) from one 32-bit word: floor(x * n / 2^32), no rejection. */
uint32_t orc_bounded(uint32_t x, uint32_t n) { return (uint32_t)(((uint64_t)x * n) >> 32); }

/* Uniform in [0,1) with 24 bits, exact in binary32. */
float orc_uniform24(uint32_t x) { return (float)(x >> 8) * (1.0f / 16777216.0f); }

/* i-th 32-bit draw of the reset stream of (seed, env, episode): word i%4 of the
 * block whose counter is (i/4, env, episode, 0). */
static uint32_t reset_draw(uint64_t seed, uint32_t env, uint32_t episode, uint32_t i) {
  uint32_t ctr[4] = {i / 4u, env, episode, 0u};
  uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32) ^ ORC_DOMAIN_RESET};
  uint32_t out[4];
  orc_philox4x32_10(ctr, key, out);
  return out[i % 4u];
}

/* Uniform for the action of `agent` in `env` at global step t_global (word 0 of
 * the block with counter (t_global, env, agent, 0)). */
float orc_action_uniform(uint64_t seed, uint32_t t_global, uint32_t env, uint32_t agent) {
  uint32_t ctr[4] = {t_global, env, agent, 0u};
  uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32) ^ ORC_DOMAIN_ACTION};
  uint32_t out[4];
  orc_philox4x32_10(ctr, key, out);
  return orc_uniform24(out[0]);
}

/* ------------------------------------------------------------------------- */
/* Reset.  Draw order: N agent levels (1 + U{0..Lmax-1}); F food levels        */
/* (1 + U{0..S-1}, S = sum of the agent levels just drawn); then N+F position  */
/* draws, agents first: draw k picks r in [0, G*G-k) and the entity takes the  */
/* r-th cell, in row-major order, not yet taken by an earlier entity.          */
/* ------------------------------------------------------------------------- */
void orc_env_reset(const orc_config_t *cfg, uint64_t seed, int32_t env, int32_t episode,
                   orc_env_state_t *s) {
  const int G = cfg->grid, N = cfg->n_agents, F = cfg->n_food;
  memset(s, 0, sizeof(*s));
  s->episode = episode;
  s->step = 0;
  uint32_t draw = 0;
  int level_sum = 0;
  for (int n = 0; n < N; ++n) {
    s->agent_level[n] =
        1 + (int32_t)orc_bounded(reset_draw(seed, (uint32_t)env, (uint32_t)episode, draw++),
                                 (uint32_t)cfg->max_agent_level);
    level_sum += s->agent_level[n];
  }
  s->total_food_level = 0;
  for (int f = 0; f < F; ++f) {
    s->food_level[f] =
        1 + (int32_t)orc_bounded(reset_draw(seed, (uint32_t)env, (uint32_t)episode, draw++),
                                 (uint32_t)level_sum);
    s->total_food_level += s->food_level[f];
  }
  uint8_t *taken = (uint8_t *)calloc((size_t)G * G, 1);
  for (int k = 0; k < N + F; ++k) {
    uint32_t r = orc_bounded(reset_draw(seed, (uint32_t)env, (uint32_t)episode, draw++),
                             (uint32_t)(G * G - k));
    int cell = -1;
    uint32_t seen_free = 0;
    for (int i = 0; i < G * G; ++i) {
      if (taken[i]) continue;
      if (seen_free == r) { cell = i; break; }
      ++seen_free;
    }
    taken[cell] = 1;
    if (k < N) { s->agent_r[k] = cell / G; s->agent_c[k] = cell % G; }
    else { s->food_r[k - N] = cell / G; s->food_c[k - N] = cell % G; }
  }
  free(taken);
}

/* ------------------------------------------------------------------------- */
/* Observation of one agent: egocentric (2R+1)^2 window in three channel       */
/* planes (agent level, food level, wall), then own level, step/cap, and the   */
/* one-hot agent id.  Entry ch*W*W + (dy+R)*W + (dx+R) describes cell          */
/* (r+dy, c+dx).  Cells outside the G x G playable area are wall.              */
/* ------------------------------------------------------------------------- */
void orc_env_observe(const orc_config_t *cfg, const orc_env_state_t *s, int32_t agent, float *obs) {
  const int G = cfg->grid, N = cfg->n_agents, F = cfg->n_food, R = cfg->view_radius;
  const int W = 2 * R + 1;
  const int D = orc_obs_dim(cfg);
  for (int i = 0; i < D; ++i) obs[i] = 0.0f;
  const int r0 = s->agent_r[agent], c0 = s->agent_c[agent];
  for (int dy = -R; dy <= R; ++dy) {
    for (int dx = -R; dx <= R; ++dx) {
      const int rr = r0 + dy, cc = c0 + dx;
      const int idx = (dy + R) * W + (dx + R);
      if (rr < 0 || rr >= G || cc < 0 || cc >= G) {
        obs[2 * W * W + idx] = 1.0f;
        continue;
      }
      for (int n = 0; n < N; ++n)
        if (s->agent_r[n] == rr && s->agent_c[n] == cc) obs[idx] = (float)s->agent_level[n];
      for (int f = 0; f < F; ++f)
        if (s->food_level[f] > 0 && s->food_r[f] == rr && s->food_c[f] == cc)
          obs[W * W + idx] = (float)s->food_level[f];
    }
  }
  obs[3 * W * W] = (float)s->agent_level[agent];
  obs[3 * W * W + 1] = (float)s->step / (float)cfg->episode_cap;
  obs[3 * W * W + 2 + agent] = 1.0f;
}

/* ------------------------------------------------------------------------- */
/* Transition.  Actions: 0 noop, 1 up (r-1), 2 down (r+1), 3 left (c-1),       */
/* 4 right (c+1), 5 load.  All decisions are taken on the start-of-step state: */
/* a move is cancelled if its target cell is outside the grid, holds a food    */
/* that is still present, is the current cell of another agent, or is also the */
/* target of another moving agent.  A present food is collected when the       */
/* levels of the loading agents 4-adjacent to it sum to at least its level.    */
/* All agents receive (sum of levels collected this step) / (total food level  */
/* at reset), one binary32 division.  Then step += 1 and the episode is done   */
/* when no food is left or step has reached the cap.  No reset happens here.   */
/* ------------------------------------------------------------------------- */
void orc_env_step(const orc_config_t *cfg, orc_env_state_t *s, const int32_t *actions,
                  float *reward, uint8_t *done) {
  const int G = cfg->grid, N = cfg->n_agents, F = cfg->n_food;
  static const int dr[ORC_N_ACTIONS] = {0, -1, 1, 0, 0, 0};
  static const int dc[ORC_N_ACTIONS] = {0, 0, 0, -1, 1, 0};
  int moving[ORC_MAX_AGENTS], tr[ORC_MAX_AGENTS], tc[ORC_MAX_AGENTS], ok[ORC_MAX_AGENTS];
  for (int n = 0; n < N; ++n) {
    const int a = actions[n];
    moving[n] = (a >= 1 && a <= 4);
    tr[n] = s->agent_r[n] + (moving[n] ? dr[a] : 0);
    tc[n] = s->agent_c[n] + (moving[n] ? dc[a] : 0);
  }
  for (int n = 0; n < N; ++n) {
    ok[n] = moving[n];
    if (!moving[n]) continue;
    if (tr[n] < 0 || tr[n] >= G || tc[n] < 0 || tc[n] >= G) ok[n] = 0;
    for (int f = 0; f < F; ++f)
      if (s->food_level[f] > 0 && s->food_r[f] == tr[n] && s->food_c[f] == tc[n]) ok[n] = 0;
    for (int m = 0; m < N; ++m) {
      if (m == n) continue;
      if (s->agent_r[m] == tr[n] && s->agent_c[m] == tc[n]) ok[n] = 0;
      if (moving[m] && tr[m] == tr[n] && tc[m] == tc[n]) ok[n] = 0;
    }
  }
  int collected_sum = 0;
  int collected[ORC_MAX_FOOD];
  for (int f = 0; f < F; ++f) {
    collected[f] = 0;
    if (s->food_level[f] <= 0) continue;
    int load_sum = 0;
    for (int n = 0; n < N; ++n) {
      if (actions[n] != 5) continue;
      const int dist = abs(s->agent_r[n] - s->food_r[f]) + abs(s->agent_c[n] - s->food_c[f]);
      if (dist == 1) load_sum += s->agent_level[n];
    }
    if (load_sum >= s->food_level[f]) { collected[f] = 1; collected_sum += s->food_level[f]; }
  }
  for (int n = 0; n < N; ++n)
    if (ok[n]) { s->agent_r[n] = tr[n]; s->agent_c[n] = tc[n]; }
  for (int f = 0; f < F; ++f)
    if (collected[f]) s->food_level[f] = 0;
  *reward = (collected_sum > 0) ? (float)collected_sum / (float)s->total_food_level : 0.0f;
  s->step += 1;
  int food_left = 0;
  for (int f = 0; f < F; ++f) food_left += (s->food_level[f] > 0);
  *done = (uint8_t)((food_left == 0) || (s->step >= cfg->episode_cap));
}

/* ------------------------------------------------------------------------- */
/* Warehouse gridworld (the second workload family; Section 4, "Multi-Robot     */
/* Warehouse": robots fetch requested shelves, and the variant the report       */
/* trains on ends the episode on collisions).  The report gives no rules; the   */
/* ones below were written for this library, sized so that observations,        */
/* actions and networks are those of the foraging workloads.                    */
/*                                                                             */
/* State (in the fields of orc_env_state_t): robot n at (agent_r, agent_c),     */
/* agent_level[n] = 0 when empty-handed, 1 + f while it carries shelf f;        */
/* shelf f at (food_r, food_c) -- a carried shelf is at its carrier's cell --   */
/* food_level[f] = 1 idle, 2 requested; total_food_level counts the deliveries  */
/* of the episode.  Row 0 is the delivery row.  floor(F/2) shelves (at least    */
/* one) are requested at all times.                                             */
/*                                                                             */
/* Reset (draws i = 0, 1, ... of the episode's reset stream): F shelf cells:    */
/* draw k picks r in [0, (G-1)*G - k) and shelf k takes the r-th cell, in       */
/* row-major order over rows 1..G-1, that no earlier shelf took; N robot cells: */
/* draw picks r in [0, G*G - F - n) and robot n takes the r-th cell of the      */
/* whole grid that holds neither a shelf nor an earlier robot; then the         */
/* requests: draw k picks r in [0, F - k) and the r-th still idle shelf in      */
/* index order becomes requested.                                               */
/* ------------------------------------------------------------------------- */
static int wh_requests(const orc_config_t *cfg) { return cfg->n_food / 2 > 0 ? cfg->n_food / 2 : 1; }

void orc_wh_reset(const orc_config_t *cfg, uint64_t seed, int32_t env, int32_t episode, orc_env_state_t *s) {
  const int G = cfg->grid, N = cfg->n_agents, F = cfg->n_food;
  memset(s, 0, sizeof(*s));
  s->episode = episode;
  uint32_t draw = 0;
  uint8_t *taken = (uint8_t *)calloc((size_t)G * G, 1);
  for (int k = 0; k < F; ++k) {
    uint32_t r = orc_bounded(reset_draw(seed, (uint32_t)env, (uint32_t)episode, draw++), (uint32_t)((G - 1) * G - k));
    for (int i = G; i < G * G; ++i) {  /* rows 1 .. G-1 */
      if (taken[i]) continue;
      if (r == 0) { taken[i] = 1; s->food_r[k] = i / G; s->food_c[k] = i % G; break; }
      --r;
    }
    s->food_level[k] = 1;
  }
  for (int n = 0; n < N; ++n) {
    uint32_t r = orc_bounded(reset_draw(seed, (uint32_t)env, (uint32_t)episode, draw++), (uint32_t)(G * G - F - n));
    for (int i = 0; i < G * G; ++i) {
      if (taken[i]) continue;
      if (r == 0) { taken[i] = 1; s->agent_r[n] = i / G; s->agent_c[n] = i % G; break; }
      --r;
    }
    s->agent_level[n] = 0;
  }
  free(taken);
  for (int k = 0; k < wh_requests(cfg); ++k) {
    uint32_t r = orc_bounded(reset_draw(seed, (uint32_t)env, (uint32_t)episode, draw++), (uint32_t)(F - k));
    for (int f = 0; f < F; ++f) {
      if (s->food_level[f] != 1) continue;
      if (r == 0) { s->food_level[f] = 2; break; }
      --r;
    }
  }
}

/* Observation of robot `agent`: the same three 5x5 planes and scalars as the   */
/* foraging workload, with these meanings: plane 0: 1 at an empty-handed        */
/* robot's cell, 2 at a carrying robot's (own cell included); plane 1: 1 at an  */
/* idle shelf's cell, 2 at a requested shelf's (on the ground or carried);      */
/* plane 2: 1 outside the grid, 0.5 on the delivery row; then 1 or 2 for the    */
/* robot itself, step/cap, one-hot id.                                          */
void orc_wh_observe(const orc_config_t *cfg, const orc_env_state_t *s, int32_t agent, float *obs) {
  const int G = cfg->grid, N = cfg->n_agents, F = cfg->n_food, R = cfg->view_radius;
  const int W = 2 * R + 1, D = orc_obs_dim(cfg);
  for (int i = 0; i < D; ++i) obs[i] = 0.0f;
  const int r0 = s->agent_r[agent], c0 = s->agent_c[agent];
  for (int dy = -R; dy <= R; ++dy) {
    for (int dx = -R; dx <= R; ++dx) {
      const int rr = r0 + dy, cc = c0 + dx, idx = (dy + R) * W + (dx + R);
      if (rr < 0 || rr >= G || cc < 0 || cc >= G) { obs[2 * W * W + idx] = 1.0f; continue; }
      if (rr == 0) obs[2 * W * W + idx] = 0.5f;
      for (int n = 0; n < N; ++n)
        if (s->agent_r[n] == rr && s->agent_c[n] == cc) obs[idx] = s->agent_level[n] > 0 ? 2.0f : 1.0f;
      for (int f = 0; f < F; ++f)
        if (s->food_r[f] == rr && s->food_c[f] == cc) obs[W * W + idx] = (float)s->food_level[f];
    }
  }
  obs[3 * W * W] = s->agent_level[agent] > 0 ? 2.0f : 1.0f;
  obs[3 * W * W + 1] = (float)s->step / (float)cfg->episode_cap;
  obs[3 * W * W + 2 + agent] = 1.0f;
}

/* Transition, all decisions on the start-of-step state.                        */
/*  Moves (actions 1..4): cancelled if the target is outside the grid, is       */
/*   another robot's current cell, is another mover's target, or -- for a robot */
/*   that carries a shelf -- holds a shelf standing on the ground.  The second  */
/*   and third reasons are robot conflicts.  A carried shelf moves with its     */
/*   robot; an empty-handed robot may pass under shelves.                       */
/*  Action 5: an empty-handed robot standing under a shelf on the ground picks  */
/*   it up; a carrying robot outside the delivery row puts its shelf down.      */
/*  Delivery: a carrying robot whose cell after the moves is in the delivery    */
/*   row, with a requested shelf, delivers it: the shelf becomes idle (and      */
/*   stays on the robot).  For the deliveries in robot order, the d-th one      */
/*   (d = 0, 1, ...) draws the replacement request: word 0 of the Philox block  */
/*   with counter (d, env, episode, step) under the request key picks r in      */
/*   [0, n) and the r-th of the n shelves that are idle and were not delivered  */
/*   in this step, in index order, becomes requested.                           */
/*  Reward: the number of deliveries of the step, to every robot.  step += 1;   */
/*  done when the cap is reached, or (env_kind 2) when a robot conflict         */
/*  cancelled a move in this step.  No reset happens here.                      */
void orc_wh_step(const orc_config_t *cfg, uint64_t seed, int32_t env, orc_env_state_t *s, const int32_t *actions,
                 float *reward, uint8_t *done) {
  const int G = cfg->grid, N = cfg->n_agents, F = cfg->n_food;
  static const int dr[ORC_N_ACTIONS] = {0, -1, 1, 0, 0, 0};
  static const int dc[ORC_N_ACTIONS] = {0, 0, 0, -1, 1, 0};
  int moving[ORC_MAX_AGENTS], tr[ORC_MAX_AGENTS], tc[ORC_MAX_AGENTS], ok[ORC_MAX_AGENTS];
  int carried[ORC_MAX_FOOD]; /* shelf f is on a robot at the start of the step */
  for (int f = 0; f < F; ++f) carried[f] = 0;
  for (int n = 0; n < N; ++n)
    if (s->agent_level[n] > 0) carried[s->agent_level[n] - 1] = 1;
  for (int n = 0; n < N; ++n) {
    const int a = actions[n];
    moving[n] = (a >= 1 && a <= 4);
    tr[n] = s->agent_r[n] + (moving[n] ? dr[a] : 0);
    tc[n] = s->agent_c[n] + (moving[n] ? dc[a] : 0);
  }
  int conflict = 0;
  for (int n = 0; n < N; ++n) {
    ok[n] = moving[n];
    if (!moving[n]) continue;
    if (tr[n] < 0 || tr[n] >= G || tc[n] < 0 || tc[n] >= G) ok[n] = 0;
    for (int m = 0; m < N; ++m) {
      if (m == n) continue;
      if (s->agent_r[m] == tr[n] && s->agent_c[m] == tc[n]) { ok[n] = 0; conflict = 1; }
      if (moving[m] && tr[m] == tr[n] && tc[m] == tc[n]) { ok[n] = 0; conflict = 1; }
    }
    if (s->agent_level[n] > 0)
      for (int f = 0; f < F; ++f)
        if (!carried[f] && s->food_r[f] == tr[n] && s->food_c[f] == tc[n]) ok[n] = 0;
  }
  /* pick up / put down, at the start-of-step cell */
  int new_carry[ORC_MAX_AGENTS];
  for (int n = 0; n < N; ++n) {
    new_carry[n] = s->agent_level[n];
    if (actions[n] != 5) continue;
    if (s->agent_level[n] == 0) {
      for (int f = 0; f < F; ++f)
        if (!carried[f] && s->food_r[f] == s->agent_r[n] && s->food_c[f] == s->agent_c[n]) new_carry[n] = 1 + f;
    } else if (s->agent_r[n] != 0) {
      new_carry[n] = 0;
    }
  }
  for (int n = 0; n < N; ++n) {
    s->agent_level[n] = new_carry[n];
    if (ok[n]) {
      s->agent_r[n] = tr[n]; s->agent_c[n] = tc[n];
      if (s->agent_level[n] > 0) { s->food_r[s->agent_level[n] - 1] = tr[n]; s->food_c[s->agent_level[n] - 1] = tc[n]; }
    }
  }
  int delivered_now[ORC_MAX_FOOD], d = 0;
  for (int f = 0; f < F; ++f) delivered_now[f] = 0;
  for (int n = 0; n < N; ++n) {
    const int f = s->agent_level[n] - 1;
    if (f >= 0 && s->agent_r[n] == 0 && s->food_level[f] == 2) { s->food_level[f] = 1; delivered_now[f] = 1; ++d; }
  }
  for (int k = 0; k < d; ++k) {
    int n_idle = 0;
    for (int f = 0; f < F; ++f) n_idle += (s->food_level[f] == 1 && !delivered_now[f]);
    if (n_idle == 0) break;
    uint32_t ctr[4] = {(uint32_t)k, (uint32_t)env, (uint32_t)s->episode, (uint32_t)s->step};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32) ^ ORC_DOMAIN_REQUEST};
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    uint32_t r = orc_bounded(out[0], (uint32_t)n_idle);
    for (int f = 0; f < F; ++f) {
      if (s->food_level[f] != 1 || delivered_now[f]) continue;
      if (r == 0) { s->food_level[f] = 2; break; }
      --r;
    }
  }
  s->total_food_level += d;
  *reward = (float)d;
  s->step += 1;
  *done = (uint8_t)((s->step >= cfg->episode_cap) || (cfg->env_kind == 2 && conflict));
}

/* The workload family selects the environment's three routines. */
static void any_reset(const orc_config_t *cfg, uint64_t seed, int32_t env, int32_t episode, orc_env_state_t *s) {
  if (cfg->env_kind == 0) orc_env_reset(cfg, seed, env, episode, s);
  else orc_wh_reset(cfg, seed, env, episode, s);
}
static void any_observe(const orc_config_t *cfg, const orc_env_state_t *s, int32_t agent, float *obs) {
  if (cfg->env_kind == 0) orc_env_observe(cfg, s, agent, obs);
  else orc_wh_observe(cfg, s, agent, obs);
}
static void any_step(const orc_config_t *cfg, uint64_t seed, int32_t env, orc_env_state_t *s, const int32_t *actions,
                     float *reward, uint8_t *done) {
  if (cfg->env_kind == 0) orc_env_step(cfg, s, actions, reward, done);
  else orc_wh_step(cfg, seed, env, s, actions, reward, done);
}

/* ------------------------------------------------------------------------- */
/* MLP.  Dense layers follow the y = x W^T + b convention with W stored        */
/* [out][in]; ReLU after both hidden layers, linear heads.  Parameter order    */
/*   net_kind 0: W1[H][D] b1[H] W2[H][H] b2[H] Wa[6][H] ba[6] Wv[1][H] bv[1]   */
/*   net_kind 1: the actor (W1 b1 W2 b2 Wa ba) and then the critic             */
/*               C1[H][N*D] c1[H] C2[H][H] c2[H] Cv[1][H] cv[1], whose input   */
/*               is the observations of agents 0..N-1 concatenated.            */
/* emulate_bf16 != 0 rounds inputs, weights and hidden activations to bfloat16 */
/* (round to nearest even) before each product, to mirror a tensor-core path   */
/* with bf16 operands; sums stay in double and biases stay binary32.           */
/* ------------------------------------------------------------------------- */
int64_t orc_params_count(const orc_config_t *cfg) {
  const int64_t D = orc_obs_dim(cfg), H = cfg->hidden, N = cfg->n_agents;
  int64_t torso = H * D + H + H * H + H;
  int64_t actor_head = ORC_N_ACTIONS * H + ORC_N_ACTIONS;
  int64_t value_head = H + 1;
  if (cfg->net_kind == 0) return torso + actor_head + value_head;
  return torso + actor_head + (H * N * D + H + H * H + H) + value_head;
}

float orc_bf16_round(float x) {
  uint32_t u;
  memcpy(&u, &x, 4);
  if ((u & 0x7F800000u) == 0x7F800000u) return x; /* inf / nan unchanged */
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  u &= 0xFFFF0000u;
  float y;
  memcpy(&y, &u, 4);
  return y;
}

static double q(float v, int emulate_bf16) {
  return (double)(emulate_bf16 ? orc_bf16_round(v) : v);
}

/* y[o] = act(sum_k W[o][k] x[k] + b[o]); x is given in double. */
static void dense(const float *W, const float *b, const double *x, int in_dim, int out_dim,
                  int relu, int emulate_bf16, double *y) {
  for (int o = 0; o < out_dim; ++o) {
    double acc = 0.0;
    for (int k = 0; k < in_dim; ++k) acc += q(W[(size_t)o * in_dim + k], emulate_bf16) * x[k];
    acc += (double)b[o];
    if (relu && acc < 0.0) acc = 0.0;
    y[o] = acc;
  }
}

static void round_vec(double *v, int n, int emulate_bf16) {
  if (!emulate_bf16) return;
  for (int i = 0; i < n; ++i) v[i] = (double)orc_bf16_round((float)v[i]);
}

/* Forward of one environment: obs is [N][D] binary32; logits [N][6] and
 * values [N] come out in double.  For net_kind 1 the single centralised value
 * is written to all N slots. */
void orc_mlp_forward_env(const orc_config_t *cfg, const float *params, const float *obs,
                         int emulate_bf16, double *logits, double *values) {
  const int D = orc_obs_dim(cfg), H = cfg->hidden, N = cfg->n_agents;
  const float *W1 = params, *b1 = W1 + (size_t)H * D, *W2 = b1 + H, *b2 = W2 + (size_t)H * H;
  const float *Wa = b2 + H, *ba = Wa + (size_t)ORC_N_ACTIONS * H;
  const float *rest = ba + ORC_N_ACTIONS;
  double *x = (double *)malloc(sizeof(double) * (size_t)N * D);
  double *h1 = (double *)malloc(sizeof(double) * (size_t)H);
  double *h2 = (double *)malloc(sizeof(double) * (size_t)H);
  for (int i = 0; i < N * D; ++i) x[i] = q(obs[i], emulate_bf16);
  for (int n = 0; n < N; ++n) {
    dense(W1, b1, x + (size_t)n * D, D, H, 1, emulate_bf16, h1);
    round_vec(h1, H, emulate_bf16);
    dense(W2, b2, h1, H, H, 1, emulate_bf16, h2);
    round_vec(h2, H, emulate_bf16);
    dense(Wa, ba, h2, H, ORC_N_ACTIONS, 0, emulate_bf16, logits + (size_t)n * ORC_N_ACTIONS);
    if (cfg->net_kind == 0) {
      const float *Wv = rest, *bv = Wv + H;
      dense(Wv, bv, h2, H, 1, 0, emulate_bf16, values + n);
    }
  }
  if (cfg->net_kind == 1) {
    const int DC = N * D;
    const float *C1 = rest, *c1 = C1 + (size_t)H * DC, *C2 = c1 + H, *c2 = C2 + (size_t)H * H;
    const float *Cv = c2 + H, *cv = Cv + H;
    double v;
    dense(C1, c1, x, DC, H, 1, emulate_bf16, h1);
    round_vec(h1, H, emulate_bf16);
    dense(C2, c2, h1, H, H, 1, emulate_bf16, h2);
    round_vec(h2, H, emulate_bf16);
    dense(Cv, cv, h2, H, 1, 0, emulate_bf16, &v);
    for (int n = 0; n < N; ++n) values[n] = v;
  }
  free(x); free(h1); free(h2);
}

/* ------------------------------------------------------------------------- */
/* Categorical sampling by inverse CDF on the softmax of six logits:           */
/* m = max l; e_k = exp(l_k - m); S = e_0 + ... + e_5 in index order; the      */
/* action is the smallest k with u*S < e_0 + ... + e_k (5 if none), and        */
/* logp_k = l_k - m - log S.  margin = distance from u*S to the nearest        */
/* interior CDF boundary, divided by S (how close the draw was to flipping).   */
/* ------------------------------------------------------------------------- */
void orc_sample(const double *logits, float u, int32_t *action, double *logp_all, double *margin) {
  double m = logits[0];
  for (int k = 1; k < ORC_N_ACTIONS; ++k) if (logits[k] > m) m = logits[k];
  double e[ORC_N_ACTIONS], S = 0.0;
  for (int k = 0; k < ORC_N_ACTIONS; ++k) { e[k] = exp(logits[k] - m); S += e[k]; }
  const double target = (double)u * S;
  double cdf = 0.0, best = INFINITY;
  int a = ORC_N_ACTIONS - 1, found = 0;
  for (int k = 0; k < ORC_N_ACTIONS; ++k) {
    cdf += e[k];
    if (!found && target < cdf) { a = k; found = 1; }
    if (k < ORC_N_ACTIONS - 1) { double d = fabs(target - cdf); if (d < best) best = d; }
  }
  *action = a;
  for (int k = 0; k < ORC_N_ACTIONS; ++k) logp_all[k] = logits[k] - m - log(S);
  if (margin) *margin = best / S;
}

/* ------------------------------------------------------------------------- */
/* Rollout of n_local environments for T steps.  Per step and environment:     */
/* observe -> MLP -> sample -> transition -> (reset when done).  The terminal  */
/* observation is dropped: after a done the next row shows the new episode.    */
/* values[T] is the critic on the observation that follows the last step.      */
/*                                                                             */
/* env_ids[i] is the global environment index (it keys Philox); its data sit   */
/* at array position pos0 + i of arrays whose environment extent is E_arr.     */
/* forced_actions (same layout as actions) replaces the sampled action when    */
/* given ("teacher forcing"); own_actions always receives the oracle's own     */
/* sample.  compute_mlp == 0 skips the network (forced_actions required) and   */
/* leaves logits/values/logp/own_actions/margin untouched.  Any output         */
/* pointer may be NULL.  Returns 0, or -1 on bad arguments.                    */
/* ------------------------------------------------------------------------- */
int orc_rollout(const orc_config_t *cfg, uint64_t seed, const float *params, int emulate_bf16,
                int compute_mlp, int32_t n_local, const int32_t *env_ids, int32_t E_arr,
                int32_t pos0, int32_t T, uint32_t t_global0, orc_env_state_t *states,
                const int32_t *forced_actions, float *obs, int32_t *actions, int32_t *own_actions,
                double *logp, double *values, float *rewards, uint8_t *dones, double *logits,
                double *margin) {
  const int N = cfg->n_agents, D = orc_obs_dim(cfg);
  if (N > ORC_MAX_AGENTS || cfg->n_food > ORC_MAX_FOOD) return -1;
  if (!compute_mlp && !forced_actions) return -1;
  if (compute_mlp && !params) return -1;
  float *o = (float *)malloc(sizeof(float) * (size_t)N * D);
  double lg[ORC_MAX_AGENTS * ORC_N_ACTIONS], val[ORC_MAX_AGENTS], lp[ORC_N_ACTIONS];
  int32_t act[ORC_MAX_AGENTS];
  for (int i = 0; i < n_local; ++i) {
    const int32_t env = env_ids[i];
    const size_t p = (size_t)pos0 + (size_t)i;
    orc_env_state_t *s = &states[i];
    for (int t = 0; t <= T; ++t) {
      const size_t row0 = ((size_t)t * E_arr + p) * N; /* first agent row of (t, env) */
      if (obs || compute_mlp)
        for (int n = 0; n < N; ++n) any_observe(cfg, s, n, o + (size_t)n * D);
      if (t < T && obs) memcpy(obs + row0 * D, o, sizeof(float) * (size_t)N * D);
      if (compute_mlp) {
        orc_mlp_forward_env(cfg, params, o, emulate_bf16, lg, val);
        if (values) for (int n = 0; n < N; ++n) values[row0 + n] = val[n];
      }
      if (t == T) break;
      for (int n = 0; n < N; ++n) {
        int32_t own = 0;
        if (compute_mlp) {
          double mg;
          const float u = orc_action_uniform(seed, t_global0 + (uint32_t)t, (uint32_t)env, (uint32_t)n);
          orc_sample(lg + n * ORC_N_ACTIONS, u, &own, lp, &mg);
          if (own_actions) own_actions[row0 + n] = own;
          if (margin) margin[row0 + n] = mg;
          if (logits)
            for (int k = 0; k < ORC_N_ACTIONS; ++k)
              logits[(row0 + n) * ORC_N_ACTIONS + k] = lg[n * ORC_N_ACTIONS + k];
        }
        act[n] = forced_actions ? forced_actions[row0 + n] : own;
        if (act[n] < 0 || act[n] >= ORC_N_ACTIONS) { free(o); return -1; }
        if (actions) actions[row0 + n] = act[n];
        if (compute_mlp && logp) logp[row0 + n] = lp[act[n]];
      }
      float reward;
      uint8_t done;
      any_step(cfg, seed, env, s, act, &reward, &done);
      if (rewards) for (int n = 0; n < N; ++n) rewards[row0 + n] = reward;
      if (dones) dones[(size_t)t * E_arr + p] = done;
      if (done) any_reset(cfg, seed, env, s->episode + 1, s);
    }
  }
  free(o);
  return 0;
}

/* ------------------------------------------------------------------------- */
/* Recurrent policy (Section 2: every system comes in a feed-forward and a      */
/* recurrent version; Section 4: the LBF and SMAX results are recurrent).  The  */
/* report names no cell and no sizes.  Reading taken here: the observation is   */
/* embedded by one dense ReLU layer, a gated recurrent unit (Cho et al. 2014)   */
/* of the same width carries one hidden vector per agent, and the two heads     */
/* read the new hidden vector:                                                  */
/*   e  = relu(W1 x + b1)                                                       */
/*   r  = sigma(Wir e + bir + Whr h + bhr)                                      */
/*   z  = sigma(Wiz e + biz + Whz h + bhz)                                      */
/*   n  = tanh(Win e + bin + r * (Whn h + bhn))                                 */
/*   h' = (1 - z) * n + z * h                                                   */
/*   logits = Wa h' + ba,  value = Wv h' + bv.                                  */
/* Parameter order: W1[H][D] b1[H]  Wih[3H][H] bih[3H]  Whh[3H][H] bhh[3H]      */
/* Wa[6][H] ba[6]  Wv[1][H] bv[1]; the three H-row blocks of Wih/Whh/bih/bhh are */
/* the gates r, z, n in that order.  h is zero at the start of every episode:   */
/* after a step that ends the episode every agent of that environment goes on   */
/* with h = 0.  With emulate_bf16 the operands of every product (x, e, h and    */
/* the weights) are rounded to bf16, the gate arithmetic is not, and the        */
/* carried state itself is the bf16-rounded h' (it is what the next step        */
/* multiplies and blends).                                                      */
/* ------------------------------------------------------------------------- */
int64_t orc_rec_params_count(const orc_config_t *cfg) {
  const int64_t D = orc_obs_dim(cfg), H = cfg->hidden;
  return H * D + H + 2 * (3 * H * H + 3 * H) + ORC_N_ACTIONS * H + ORC_N_ACTIONS + H + 1;
}

static double sigmoid(double v) { return 1.0 / (1.0 + exp(-v)); }

/* One environment, one step: obs [N][D] binary32, h [N][H] in and out (double). */
void orc_rec_forward_env(const orc_config_t *cfg, const float *params, const float *obs, double *h,
                         int emulate_bf16, double *logits, double *values) {
  const int D = orc_obs_dim(cfg), H = cfg->hidden, N = cfg->n_agents;
  const float *W1 = params, *b1 = W1 + (size_t)H * D;
  const float *Wih = b1 + H, *bih = Wih + (size_t)3 * H * H;
  const float *Whh = bih + 3 * H, *bhh = Whh + (size_t)3 * H * H;
  const float *Wa = bhh + 3 * H, *ba = Wa + (size_t)ORC_N_ACTIONS * H, *Wv = ba + ORC_N_ACTIONS, *bv = Wv + H;
  double *x = (double *)malloc(sizeof(double) * (size_t)D);
  double *e = (double *)malloc(sizeof(double) * (size_t)H);
  double *gi = (double *)malloc(sizeof(double) * (size_t)3 * H);
  double *gh = (double *)malloc(sizeof(double) * (size_t)3 * H);
  for (int n = 0; n < N; ++n) {
    double *hn = h + (size_t)n * H;
    round_vec(hn, H, emulate_bf16); /* a carried state already is a bf16 number; any other input becomes one */
    for (int k = 0; k < D; ++k) x[k] = q(obs[(size_t)n * D + k], emulate_bf16);
    dense(W1, b1, x, D, H, 1, emulate_bf16, e);
    round_vec(e, H, emulate_bf16);
    dense(Wih, bih, e, H, 3 * H, 0, emulate_bf16, gi);   /* input part of the three gates, biases included  */
    dense(Whh, bhh, hn, H, 3 * H, 0, emulate_bf16, gh);  /* hidden part of the three gates, biases included */
    for (int j = 0; j < H; ++j) {
      const double r = sigmoid(gi[j] + gh[j]);
      const double z = sigmoid(gi[H + j] + gh[H + j]);
      const double c = tanh(gi[2 * H + j] + r * gh[2 * H + j]);
      hn[j] = (1.0 - z) * c + z * hn[j];
    }
    round_vec(hn, H, emulate_bf16);
    dense(Wa, ba, hn, H, ORC_N_ACTIONS, 0, emulate_bf16, logits + (size_t)n * ORC_N_ACTIONS);
    dense(Wv, bv, hn, H, 1, 0, emulate_bf16, values + n);
  }
  free(x); free(e); free(gi); free(gh);
}

/* The rollout loop of orc_rollout with the recurrent policy.  `hidden` is        */
/* [n_local][N][H] (double): the state every listed environment's agents enter    */
/* the first step with; on return, the state they would enter step T with.  The   */
/* bootstrap row values[T] is the value head on the hidden vector after one more  */
/* cell update on the observation that follows the last step; that update is not  */
/* kept (the next call repeats it on the same observation and state).             */
int orc_rollout_rec(const orc_config_t *cfg, uint64_t seed, const float *params, int emulate_bf16,
                    int32_t n_local, const int32_t *env_ids, int32_t T, uint32_t t_global0,
                    orc_env_state_t *states, double *hidden, const int32_t *forced_actions, float *obs,
                    int32_t *actions, int32_t *own_actions, double *logp, double *values, float *rewards,
                    uint8_t *dones, double *logits, double *margin) {
  const int N = cfg->n_agents, D = orc_obs_dim(cfg), H = cfg->hidden;
  if (N > ORC_MAX_AGENTS || cfg->n_food > ORC_MAX_FOOD || !params || !hidden) return -1;
  float *o = (float *)malloc(sizeof(float) * (size_t)N * D);
  double *hb = (double *)malloc(sizeof(double) * (size_t)N * H);
  double lg[ORC_MAX_AGENTS * ORC_N_ACTIONS], val[ORC_MAX_AGENTS], lp[ORC_N_ACTIONS];
  int32_t act[ORC_MAX_AGENTS];
  for (int i = 0; i < n_local; ++i) {
    const int32_t env = env_ids[i];
    orc_env_state_t *s = &states[i];
    double *h = hidden + (size_t)i * N * H;
    for (int t = 0; t <= T; ++t) {
      const size_t row0 = ((size_t)t * n_local + (size_t)i) * N;
      for (int n = 0; n < N; ++n) any_observe(cfg, s, n, o + (size_t)n * D);
      if (t < T && obs) memcpy(obs + row0 * D, o, sizeof(float) * (size_t)N * D);
      if (t == T) {  /* bootstrap: on a copy of the state */
        memcpy(hb, h, sizeof(double) * (size_t)N * H);
        orc_rec_forward_env(cfg, params, o, hb, emulate_bf16, lg, val);
        if (values) for (int n = 0; n < N; ++n) values[row0 + n] = val[n];
        break;
      }
      orc_rec_forward_env(cfg, params, o, h, emulate_bf16, lg, val);
      if (values) for (int n = 0; n < N; ++n) values[row0 + n] = val[n];
      for (int n = 0; n < N; ++n) {
        int32_t own = 0;
        double mg;
        const float u = orc_action_uniform(seed, t_global0 + (uint32_t)t, (uint32_t)env, (uint32_t)n);
        orc_sample(lg + n * ORC_N_ACTIONS, u, &own, lp, &mg);
        if (own_actions) own_actions[row0 + n] = own;
        if (margin) margin[row0 + n] = mg;
        if (logits)
          for (int k = 0; k < ORC_N_ACTIONS; ++k) logits[(row0 + n) * ORC_N_ACTIONS + k] = lg[n * ORC_N_ACTIONS + k];
        act[n] = forced_actions ? forced_actions[row0 + n] : own;
        if (act[n] < 0 || act[n] >= ORC_N_ACTIONS) { free(o); free(hb); return -1; }
        if (actions) actions[row0 + n] = act[n];
        if (logp) logp[row0 + n] = lp[act[n]];
      }
      float reward;
      uint8_t done;
      any_step(cfg, seed, env, s, act, &reward, &done);
      if (rewards) for (int n = 0; n < N; ++n) rewards[row0 + n] = reward;
      if (dones) dones[(size_t)t * n_local + i] = done;
      if (done) {
        any_reset(cfg, seed, env, s->episode + 1, s);
        for (int k = 0; k < N * H; ++k) h[k] = 0.0;  /* a new episode starts without memory */
      }
    }
  }
  free(o); free(hb);
  return 0;
}

/* ------------------------------------------------------------------------- */
/* Evaluation block (Section 2, "Multi-device training with easy checkpointing */
/* and logging": training is interleaved with blocks that run the current      */
/* policy and report how its episodes went).  The report gives no more than    */
/* that; the reading taken here: T steps of the same loop as the rollout       */
/* (observe, actor forward, act, transition, auto-reset) with no trajectory    */
/* kept.  The action is the arg max of the six logits (lowest index on a tie)  */
/* when `greedy`, else the rollout's Philox inverse-CDF draw.  Per environment */
/* three sums over the episodes that END inside the block:                     */
/*   ep_count  how many ended,                                                 */
/*   ret_sum   the sum of their returns; an episode's return is the sum of its */
/*             (shared) step rewards received inside the block, accumulated in */
/*             binary32 in step order, and the returns are added to ret_sum in */
/*             binary32 in the order the episodes end,                         */
/*   len_sum   the sum of their lengths in steps inside the block.             */
/* An episode still running when the block ends is not counted.  Arrays are    */
/* indexed by position in env_ids; forced_actions / actions / logits are       */
/* [T][n_local][N](x6), any of them may be NULL.                               */
/* ------------------------------------------------------------------------- */
int orc_evaluate(const orc_config_t *cfg, uint64_t seed, const float *params, int emulate_bf16,
                 int32_t n_local, const int32_t *env_ids, int32_t T, uint32_t t_global0,
                 orc_env_state_t *states, const int32_t *forced_actions, int greedy,
                 int32_t *ep_count, float *ret_sum, int32_t *len_sum, int32_t *actions,
                 double *logits) {
  const int N = cfg->n_agents, D = orc_obs_dim(cfg);
  if (N > ORC_MAX_AGENTS || cfg->n_food > ORC_MAX_FOOD || !params) return -1;
  float *o = (float *)malloc(sizeof(float) * (size_t)N * D);
  double lg[ORC_MAX_AGENTS * ORC_N_ACTIONS], val[ORC_MAX_AGENTS], lp[ORC_N_ACTIONS];
  int32_t act[ORC_MAX_AGENTS];
  for (int i = 0; i < n_local; ++i) {
    const int32_t env = env_ids[i];
    orc_env_state_t *s = &states[i];
    float running = 0.0f; /* return of the episode in progress */
    int32_t length = 0;   /* its steps so far                  */
    ep_count[i] = 0; ret_sum[i] = 0.0f; len_sum[i] = 0;
    for (int t = 0; t < T; ++t) {
      const size_t row0 = ((size_t)t * n_local + (size_t)i) * N;
      for (int n = 0; n < N; ++n) any_observe(cfg, s, n, o + (size_t)n * D);
      orc_mlp_forward_env(cfg, params, o, emulate_bf16, lg, val);
      for (int n = 0; n < N; ++n) {
        const double *l = lg + n * ORC_N_ACTIONS;
        int32_t own = 0;
        if (greedy) {
          for (int k = 1; k < ORC_N_ACTIONS; ++k)
            if (l[k] > l[own]) own = k;
        } else {
          double mg;
          const float u = orc_action_uniform(seed, t_global0 + (uint32_t)t, (uint32_t)env, (uint32_t)n);
          orc_sample(l, u, &own, lp, &mg);
        }
        act[n] = forced_actions ? forced_actions[row0 + n] : own;
        if (act[n] < 0 || act[n] >= ORC_N_ACTIONS) { free(o); return -1; }
        if (actions) actions[row0 + n] = act[n];
        if (logits)
          for (int k = 0; k < ORC_N_ACTIONS; ++k) logits[(row0 + n) * ORC_N_ACTIONS + k] = l[k];
      }
      float reward;
      uint8_t done;
      any_step(cfg, seed, env, s, act, &reward, &done);
      running += reward;
      length += 1;
      if (done) {
        ep_count[i] += 1;
        ret_sum[i] += running;
        len_sum[i] += length;
        running = 0.0f;
        length = 0;
        any_reset(cfg, seed, env, s->episode + 1, s);
      }
    }
  }
  free(o);
  return 0;
}

/* ------------------------------------------------------------------------- */
/* Generalised advantage estimation over a time-major trajectory.              */
/*   delta_t = r_t + gamma * V_{t+1} * (1 - d_t) - V_t                         */
/*   A_t     = delta_t + gamma * lambda * (1 - d_t) * A_{t+1},   A_T = 0       */
/*   Ret_t   = A_t + V_t                                                       */
/* values [T+1][E][N], rewards [T][E][N], dones [T][E] (shared by the agents   */
/* of an environment).  A done cuts both the bootstrap and the trace.          */
/* ------------------------------------------------------------------------- */
void orc_gae(int32_t T, int32_t E, int32_t N, const float *values, const float *rewards,
             const uint8_t *dones, double gamma, double lambda, double *adv, double *ret) {
  const size_t M = (size_t)E * N;
  for (size_t col = 0; col < M; ++col) {
    const size_t e = col / N;
    double next_adv = 0.0;
    for (int t = T - 1; t >= 0; --t) {
      const double nd = dones[(size_t)t * E + e] ? 0.0 : 1.0;
      const double v = values[(size_t)t * M + col], vn = values[(size_t)(t + 1) * M + col];
      const double delta = (double)rewards[(size_t)t * M + col] + gamma * vn * nd - v;
      const double a = delta + gamma * lambda * nd * next_adv;
      adv[(size_t)t * M + col] = a;
      ret[(size_t)t * M + col] = a + v;
      next_adv = a;
    }
  }
}

/* The same estimator as its defining sum, O(T^2) per column:
 *   A_t = sum_{l>=0} (gamma*lambda)^l * prod_{k=t}^{t+l-1} (1 - d_k) * delta_{t+l}. */
void orc_gae_bruteforce(int32_t T, int32_t E, int32_t N, const float *values, const float *rewards,
                        const uint8_t *dones, double gamma, double lambda, double *adv) {
  const size_t M = (size_t)E * N;
  for (size_t col = 0; col < M; ++col) {
    const size_t e = col / N;
    for (int t = 0; t < T; ++t) {
      double sum = 0.0;
      for (int l = 0; t + l < T; ++l) {
        double w = pow(gamma * lambda, (double)l);
        for (int k = t; k < t + l; ++k) w *= dones[(size_t)k * E + e] ? 0.0 : 1.0;
        const int s = t + l;
        const double nd = dones[(size_t)s * E + e] ? 0.0 : 1.0;
        const double delta = (double)rewards[(size_t)s * M + col] +
                             gamma * (double)values[(size_t)(s + 1) * M + col] * nd -
                             (double)values[(size_t)s * M + col];
        sum += w * delta;
      }
      adv[(size_t)t * M + col] = sum;
    }
  }
}
