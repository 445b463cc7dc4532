// Device-side gridworld: Philox4x32-10, reset, observation and transition of a tile of
// environments whose EnvRec records live in shared memory.  Every routine is written for a
// cooperating group of `nthreads` threads (thread index `tid`); the caller puts a barrier
// between the phases.  All decisions are integer arithmetic on the start-of-step state, so the
// result does not depend on how the work is split over threads.
#pragma once
#include "common.cuh"

namespace mava {

// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplications, with the
// key advanced by two Weyl constants between rounds.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t out[4]) {
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// floor(x * n / 2^32): integer in [0, n) without rejection.
__device__ __forceinline__ uint32_t bounded(uint32_t x, uint32_t n) { return __umulhi(x, n); }

// 24-bit uniform in [0, 1), exact in binary32.
__device__ __forceinline__ float uniform24(uint32_t x) {
  return static_cast<float>(x >> 8) * (1.0f / 16777216.0f);
}

// Uniform of the action draw of (global step, env, agent): word 0 of that block.
__device__ __forceinline__ float action_uniform(const EnvParams &p, uint32_t t_global, uint32_t env,
                                                uint32_t agent) {
  uint32_t o[4];
  philox4x32_10(t_global, env, agent, 0u, p.key_lo, p.key_hi ^ kDomainAction, o);
  return uniform24(o[0]);
}

// Start of an episode: N agent levels, F food levels (1 + U{0..S-1}, S = sum of agent levels),
// then N+F distinct cells: draw k picks r in [0, G*G-k) and the entity takes the r-th cell, in
// row-major order, that no earlier entity took.  The taken cells are kept sorted in registers so
// that "skip the taken cells at or below" finds that cell.  Draw i is word i%4 of the block with
// counter (i/4, env, episode, 0).
template <int N, int F>
__device__ void env_reset(EnvRec &s, const EnvParams &p, uint32_t env, uint32_t episode) {
  constexpr int K = N + F;
  constexpr int NDRAW = 2 * K;
  constexpr int NBLK = (NDRAW + 3) / 4;
  uint32_t draws[NBLK * 4];
#pragma unroll
  for (int b = 0; b < NBLK; ++b)
    philox4x32_10(static_cast<uint32_t>(b), env, episode, 0u, p.key_lo, p.key_hi ^ kDomainReset,
                  &draws[4 * b]);
  int level_sum = 0;
#pragma unroll
  for (int n = 0; n < N; ++n) {
    const int l = 1 + static_cast<int>(bounded(draws[n], static_cast<uint32_t>(p.max_level)));
    s.al[n] = static_cast<uint8_t>(l);
    level_sum += l;
  }
  int total = 0;
#pragma unroll
  for (int f = 0; f < F; ++f) {
    const int l = 1 + static_cast<int>(bounded(draws[N + f], static_cast<uint32_t>(level_sum)));
    s.fl[f] = static_cast<uint8_t>(l);
    total += l;
  }
  const int G = p.grid;
  int taken[K];
#pragma unroll
  for (int k = 0; k < K; ++k) {
    int cell = static_cast<int>(bounded(draws[K + k], static_cast<uint32_t>(G * G - k)));
#pragma unroll
    for (int j = 0; j < K; ++j)
      if (j < k && taken[j] <= cell) ++cell;
    const int r = cell / G, c = cell - r * G;
    if (k < N) { s.ar[k < N ? k : 0] = static_cast<uint8_t>(r); s.ac[k < N ? k : 0] = static_cast<uint8_t>(c); }
    else { s.fr[k >= N ? k - N : 0] = static_cast<uint8_t>(r); s.fc[k >= N ? k - N : 0] = static_cast<uint8_t>(c); }
    // sorted insert of `cell`
    int carry = cell;
#pragma unroll
    for (int j = 0; j < K; ++j) {
      if (j < k) {
        if (taken[j] > carry) { const int tmp = taken[j]; taken[j] = carry; carry = tmp; }
      } else if (j == k) {
        taken[j] = carry;
      }
    }
  }
  s.step = 0;
  s.episode = static_cast<int32_t>(episode);
  s.total = total;
}

// Observation, pass A: everything that does not depend on other entities.  sink(row, j, v)
// receives element j of agent row `row` (row = local_env * N + agent).  Planes 0 and 1 are
// zero-filled here and completed by pass B.  Element layout: [0,25) agent-level plane, [25,50)
// food-level plane, [50,75) wall plane, 75 own level, 76 step/cap, 77+a one-hot agent id.
template <int N, class Sink>
__device__ __forceinline__ void observe_fill(const EnvRec *st, const EnvParams &p, int n_rows, int tid,
                                             int nthreads, Sink sink) {
  constexpr int D = kObsFixed + N;
  const int G = p.grid;
  for (int idx = tid; idx < n_rows * D; idx += nthreads) {
    const int row = idx / D, j = idx - row * D;
    const int le = row / N, a = row - le * N;
    const EnvRec &s = st[le];
    float v = 0.0f;
    if (j >= 2 * kPlane && j < 3 * kPlane) {
      const int q = j - 2 * kPlane;
      const int dy = q / kWindow - kViewRadius, dx = q % kWindow - kViewRadius;
      const int rr = static_cast<int>(s.ar[a]) + dy, cc = static_cast<int>(s.ac[a]) + dx;
      v = (rr < 0 || rr >= G || cc < 0 || cc >= G) ? 1.0f : 0.0f;
    } else if (j == 3 * kPlane) {
      v = static_cast<float>(s.al[a]);
    } else if (j == 3 * kPlane + 1) {
      v = __fdiv_rn(static_cast<float>(s.step), static_cast<float>(p.cap));
    } else if (j >= kObsFixed) {
      v = (j - kObsFixed == a) ? 1.0f : 0.0f;
    }
    sink(row, j, v);
  }
}

// Observation, pass B: every (viewer row, entity) pair writes the entity's level where it falls
// inside the viewer's window.  Entities of one environment sit on distinct cells, so no two
// writes of a row collide.
template <int N, int F, class Sink>
__device__ __forceinline__ void observe_scatter(const EnvRec *st, int n_rows, int tid, int nthreads,
                                                Sink sink) {
  constexpr int K = N + F;
  for (int idx = tid; idx < n_rows * K; idx += nthreads) {
    const int row = idx / K, k = idx - row * K;
    const int le = row / N, a = row - le * N;
    const EnvRec &s = st[le];
    int er, ec, lvl, base;
    if (k < N) { er = s.ar[k]; ec = s.ac[k]; lvl = s.al[k]; base = 0; }
    else { er = s.fr[k - N]; ec = s.fc[k - N]; lvl = s.fl[k - N]; base = kPlane; }
    const int dy = er - static_cast<int>(s.ar[a]), dx = ec - static_cast<int>(s.ac[a]);
    if (lvl > 0 && dy >= -kViewRadius && dy <= kViewRadius && dx >= -kViewRadius && dx <= kViewRadius)
      sink(row, base + (dy + kViewRadius) * kWindow + (dx + kViewRadius), static_cast<float>(lvl));
  }
}

// Sparse form of the observation of agent `a`: calls sink(j, v) for exactly the elements that can
// be non-zero (wall cells of a window that crosses the border, entities inside the window, own
// level, step/cap, the agent's one-hot slot).  Called twice on the same state -- once with the
// values and once writing zeros -- it maintains an observation row over a zero background.
template <int N, int F, class Sink>
__device__ __forceinline__ void observe_sparse(const EnvRec &s, const EnvParams &p, int a, Sink sink) {
  const int G = p.grid;
  const int r0 = s.ar[a], c0 = s.ac[a];
  if (r0 < kViewRadius || r0 >= G - kViewRadius || c0 < kViewRadius || c0 >= G - kViewRadius) {
#pragma unroll
    for (int dy = -kViewRadius; dy <= kViewRadius; ++dy) {
#pragma unroll
      for (int dx = -kViewRadius; dx <= kViewRadius; ++dx) {
        const int rr = r0 + dy, cc = c0 + dx;
        if (rr < 0 || rr >= G || cc < 0 || cc >= G)
          sink(2 * kPlane + (dy + kViewRadius) * kWindow + (dx + kViewRadius), 1.0f);
      }
    }
  }
#pragma unroll
  for (int k = 0; k < N; ++k) {
    const int dy = static_cast<int>(s.ar[k]) - r0, dx = static_cast<int>(s.ac[k]) - c0;
    if (dy >= -kViewRadius && dy <= kViewRadius && dx >= -kViewRadius && dx <= kViewRadius)
      sink((dy + kViewRadius) * kWindow + (dx + kViewRadius), static_cast<float>(s.al[k]));
  }
#pragma unroll
  for (int f = 0; f < F; ++f) {
    const int dy = static_cast<int>(s.fr[f]) - r0, dx = static_cast<int>(s.fc[f]) - c0;
    if (s.fl[f] > 0 && dy >= -kViewRadius && dy <= kViewRadius && dx >= -kViewRadius && dx <= kViewRadius)
      sink(kPlane + (dy + kViewRadius) * kWindow + (dx + kViewRadius), static_cast<float>(s.fl[f]));
  }
  sink(3 * kPlane, static_cast<float>(s.al[a]));
  sink(3 * kPlane + 1, __fdiv_rn(static_cast<float>(s.step), static_cast<float>(p.cap)));
  sink(kObsFixed + a, 1.0f);
}

// Transition, phase 1 (reads only the start-of-step state).
//   items [0, n_rows): one agent each -> new position in new_r/new_c.  A move is cancelled when
//     its target is outside the grid, holds a present food, is another agent's current cell or is
//     another mover's target.
//   items [n_rows, n_rows + n_envs*F): one food each -> collected[] = 1 when the levels of the
//     loading agents 4-adjacent to it reach its level.
// act[row] holds the action (values outside 1..5 count as noop).
template <int N, int F>
__device__ __forceinline__ void step_decide(const EnvRec *st, const EnvParams &p, const int *act,
                                            int n_envs_tile, uint8_t *new_r, uint8_t *new_c,
                                            uint8_t *collected, int tid, int nthreads) {
  const int n_rows = n_envs_tile * N;
  const int G = p.grid;
  for (int idx = tid; idx < n_rows + n_envs_tile * F; idx += nthreads) {
    if (idx < n_rows) {
      const int le = idx / N, a = idx - le * N;
      const EnvRec &s = st[le];
      const int action = act[idx];
      const int r0 = s.ar[a], c0 = s.ac[a];
      const bool moving = action >= 1 && action <= 4;
      const int tr = r0 + (action == 2) - (action == 1), tc = c0 + (action == 4) - (action == 3);
      bool ok = moving && tr >= 0 && tr < G && tc >= 0 && tc < G;
#pragma unroll
      for (int f = 0; f < F; ++f) ok = ok && !(s.fl[f] > 0 && s.fr[f] == tr && s.fc[f] == tc);
#pragma unroll
      for (int m = 0; m < N; ++m) {
        if (m == a) continue;
        const int am = act[le * N + m];
        const int mr = s.ar[m], mc = s.ac[m];
        const bool m_moving = am >= 1 && am <= 4;
        const int mtr = mr + (am == 2) - (am == 1), mtc = mc + (am == 4) - (am == 3);
        ok = ok && !(mr == tr && mc == tc) && !(m_moving && mtr == tr && mtc == tc);
      }
      new_r[idx] = static_cast<uint8_t>(ok ? tr : r0);
      new_c[idx] = static_cast<uint8_t>(ok ? tc : c0);
    } else {
      const int q = idx - n_rows;
      const int le = q / F, f = q - le * F;
      const EnvRec &s = st[le];
      int load = 0;
#pragma unroll
      for (int n = 0; n < N; ++n) {
        const int dist = abs(static_cast<int>(s.ar[n]) - static_cast<int>(s.fr[f])) +
                         abs(static_cast<int>(s.ac[n]) - static_cast<int>(s.fc[f]));
        load += (act[le * N + n] == 5 && dist == 1) ? s.al[n] : 0;
      }
      collected[q] = static_cast<uint8_t>(s.fl[f] > 0 && load >= s.fl[f]);
    }
  }
}

// Transition, phase 2, one thread per environment: apply the moves and collections, pay the
// shared reward (collected levels / total food level, one IEEE binary32 division), advance the
// step counter, decide done (no food left, or the cap reached) and start the next episode when
// done.  Returns the reward and the done flag of local environment `le`.
template <int N, int F>
__device__ __forceinline__ void step_apply(EnvRec &s, const EnvParams &p, uint32_t env,
                                           const uint8_t *new_r, const uint8_t *new_c,
                                           const uint8_t *collected, int le, float &reward, bool &done) {
  int gained = 0, left = 0;
#pragma unroll
  for (int n = 0; n < N; ++n) { s.ar[n] = new_r[le * N + n]; s.ac[n] = new_c[le * N + n]; }
#pragma unroll
  for (int f = 0; f < F; ++f) {
    if (collected[le * F + f]) { gained += s.fl[f]; s.fl[f] = 0; }
    left += (s.fl[f] > 0);
  }
  reward = gained > 0 ? __fdiv_rn(static_cast<float>(gained), static_cast<float>(s.total)) : 0.0f;
  s.step += 1;
  done = (left == 0) || (s.step >= p.cap);
  if (done) env_reset<N, F>(s, p, env, static_cast<uint32_t>(s.episode) + 1u);
}

}  // namespace mava

// ---------------------------------------------------------------------------------------------
// Register-resident form of the same environment, for kernels where every agent row has its own
// thread and the N threads of an environment sit in adjacent lanes of one warp.  Each of those
// threads keeps a full copy of the environment (entity k packed as row | col << 8 | level << 16;
// agents first, then food, a food of level 0 is gone) and all of them apply identical integer
// updates, so the copies never diverge; what one lane decides for its own agent or food reaches
// the others by warp shuffles and ballots.
// ---------------------------------------------------------------------------------------------
namespace mava {

template <int N, int F>
struct EnvRegs {
  uint32_t ent[N + F];
  int32_t step, episode, total;
};

__device__ __forceinline__ uint32_t pack_entity(int r, int c, int level) {
  return static_cast<uint32_t>(r) | (static_cast<uint32_t>(c) << 8) | (static_cast<uint32_t>(level) << 16);
}

template <int N, int F>
__device__ __forceinline__ void load_env(EnvRegs<N, F> &s, const EnvRec &g) {
#pragma unroll
  for (int n = 0; n < N; ++n) s.ent[n] = pack_entity(g.ar[n], g.ac[n], g.al[n]);
#pragma unroll
  for (int f = 0; f < F; ++f) s.ent[N + f] = pack_entity(g.fr[f], g.fc[f], g.fl[f]);
  s.step = g.step; s.episode = g.episode; s.total = g.total;
}

template <int N, int F>
__device__ __forceinline__ void store_env(const EnvRegs<N, F> &s, EnvRec &g) {
#pragma unroll
  for (int n = 0; n < N; ++n) {
    g.ar[n] = static_cast<uint8_t>(s.ent[n]); g.ac[n] = static_cast<uint8_t>(s.ent[n] >> 8);
    g.al[n] = static_cast<uint8_t>(s.ent[n] >> 16);
  }
#pragma unroll
  for (int f = 0; f < F; ++f) {
    g.fr[f] = static_cast<uint8_t>(s.ent[N + f]); g.fc[f] = static_cast<uint8_t>(s.ent[N + f] >> 8);
    g.fl[f] = static_cast<uint8_t>(s.ent[N + f] >> 16);
  }
  g.step = s.step; g.episode = s.episode; g.total = s.total;
}

// Same draw order and placement rule as env_reset above.
template <int N, int F>
__device__ void reset_env(EnvRegs<N, F> &s, const EnvParams &p, uint32_t env, uint32_t episode) {
  constexpr int K = N + F;
  constexpr int NBLK = (2 * K + 3) / 4;
  uint32_t draws[NBLK * 4];
#pragma unroll
  for (int b = 0; b < NBLK; ++b)
    philox4x32_10(static_cast<uint32_t>(b), env, episode, 0u, p.key_lo, p.key_hi ^ kDomainReset, &draws[4 * b]);
  int level[K];
  int level_sum = 0, total = 0;
#pragma unroll
  for (int n = 0; n < N; ++n) {
    level[n] = 1 + static_cast<int>(bounded(draws[n], static_cast<uint32_t>(p.max_level)));
    level_sum += level[n];
  }
#pragma unroll
  for (int f = 0; f < F; ++f) {
    level[N + f] = 1 + static_cast<int>(bounded(draws[N + f], static_cast<uint32_t>(level_sum)));
    total += level[N + f];
  }
  const int G = p.grid;
  int taken[K];
#pragma unroll
  for (int k = 0; k < K; ++k) {
    int cell = static_cast<int>(bounded(draws[K + k], static_cast<uint32_t>(G * G - k)));
#pragma unroll
    for (int j = 0; j < K; ++j)
      if (j < k && taken[j] <= cell) ++cell;
    const int r = cell / G, c = cell - r * G;
    s.ent[k] = pack_entity(r, c, level[k]);
    int carry = cell;
#pragma unroll
    for (int j = 0; j < K; ++j) {
      if (j < k) {
        if (taken[j] > carry) { const int tmp = taken[j]; taken[j] = carry; carry = tmp; }
      } else if (j == k) {
        taken[j] = carry;
      }
    }
  }
  s.step = 0;
  s.episode = static_cast<int32_t>(episode);
  s.total = total;
}

// Non-zero observation entries of one agent (see observe_sparse for the element layout), in three
// parts that need different pieces of the state, so that different warps can produce them:
// the wall plane (from the agent's cell), the two level planes (from all entities), and the
// scalars (own level, step/cap, one-hot id).
template <class Sink>
__device__ __forceinline__ void observe_walls(int r0, int c0, int G, Sink sink) {
  bool row_out[kWindow], col_out[kWindow];
#pragma unroll
  for (int d = 0; d < kWindow; ++d) {
    row_out[d] = (r0 + d - kViewRadius < 0) || (r0 + d - kViewRadius >= G);
    col_out[d] = (c0 + d - kViewRadius < 0) || (c0 + d - kViewRadius >= G);
  }
#pragma unroll
  for (int dy = 0; dy < kWindow; ++dy)
#pragma unroll
    for (int dx = 0; dx < kWindow; ++dx)
      if (row_out[dy] || col_out[dx]) sink(2 * kPlane + dy * kWindow + dx, 1.0f);
}
template <int N, int F, class Sink>
__device__ __forceinline__ void observe_levels(const EnvRegs<N, F> &s, int r0, int c0, Sink sink) {
#pragma unroll
  for (int k = 0; k < N + F; ++k) {
    const uint32_t e = s.ent[k];
    const int dy = static_cast<int>(e & 0xFF) - r0 + kViewRadius, dx = static_cast<int>((e >> 8) & 0xFF) - c0 + kViewRadius;
    const int lvl = static_cast<int>(e >> 16);
    if (lvl > 0 && dy >= 0 && dy < kWindow && dx >= 0 && dx < kWindow)
      sink((k < N ? 0 : kPlane) + dy * kWindow + dx, static_cast<float>(lvl));
  }
}
template <class Sink>
__device__ __forceinline__ void observe_scalars(int level, int step, int cap, int ag, Sink sink) {
  sink(3 * kPlane, static_cast<float>(level));
  sink(3 * kPlane + 1, __fdiv_rn(static_cast<float>(step), static_cast<float>(cap)));
  sink(kObsFixed + ag, 1.0f);
}
template <int N, int F>
__device__ __forceinline__ uint32_t own_entity(const EnvRegs<N, F> &s, int ag) {
  uint32_t me = s.ent[0];
#pragma unroll
  for (int m = 1; m < N; ++m) me = (ag == m) ? s.ent[m] : me;
  return me;
}
template <int N, int F, class Sink>
__device__ __forceinline__ void observe_env(const EnvRegs<N, F> &s, const EnvParams &p, int ag, Sink sink) {
  const uint32_t me = own_entity(s, ag);
  const int r0 = me & 0xFF, c0 = (me >> 8) & 0xFF;
  observe_walls(r0, c0, p.grid, sink);
  observe_levels<N, F>(s, r0, c0, sink);
  observe_scalars(static_cast<int>(me >> 16), s.step, p.cap, ag, sink);
}

// One transition of the environment whose N agent threads occupy lanes [base, base + N) of this
// warp; every lane of the warp must call it (lanes without an environment pass active = false
// and base = their own lane).  `action` is this lane's action.  Same rules as step_decide /
// step_apply; returns the shared reward and the done flag, and has already started the next
// episode when done.
template <int N, int F>
__device__ __forceinline__ void step_env_warp(EnvRegs<N, F> &s, const EnvParams &p, uint32_t env, int ag, int base,
                                              bool active, int action, float &reward, bool &done) {
  constexpr unsigned kFull = 0xFFFFFFFFu;
  const int G = p.grid;
  // this lane's own agent: where it wants to go (0xFFFF: not moving, 0xFFFE: off the grid)
  uint32_t my_pos = s.ent[0] & 0xFFFFu;
#pragma unroll
  for (int m = 1; m < N; ++m) my_pos = (ag == m) ? (s.ent[m] & 0xFFFFu) : my_pos;
  uint32_t my_target;
  {
    const int r = my_pos & 0xFF, c = my_pos >> 8;
    const int tr = r + (action == 2) - (action == 1), tc = c + (action == 4) - (action == 3);
    const bool moving = action >= 1 && action <= 4;
    const bool inside = tr >= 0 && tr < G && tc >= 0 && tc < G;
    my_target = moving ? (inside ? (static_cast<uint32_t>(tr) | (static_cast<uint32_t>(tc) << 8)) : 0xFFFEu) : 0xFFFFu;
  }
  uint32_t my_new;
  uint32_t collected_mask = 0;  // bit f: food f collected
  if constexpr (N >= 3) {
    // Who tries to load, as one bit per agent of this environment; and whether another agent of this environment wants
    // the same cell: lanes with equal (environment, target) keys.  A lane that stays, leaves the grid or has no
    // environment gets a key of its own.
    const uint32_t loaders = (__ballot_sync(kFull, action == 5) >> base) & ((1u << N) - 1u);
    const uint32_t key = my_target < 0xFFFEu ? (my_target | (static_cast<uint32_t>(base) << 16)) : (0x80000000u | (threadIdx.x & 31u));
    const uint32_t same = __match_any_sync(kFull, key);
    bool ok = my_target < 0xFFFEu && (same & (same - 1u)) == 0u;  // moving, inside the grid, alone with this target
    // ... and the cell holds neither food nor an agent at the start of the step (this lane's own agent is elsewhere)
#pragma unroll
    for (int f = 0; f < F; ++f) ok = ok && !((s.ent[N + f] >> 16) != 0 && (s.ent[N + f] & 0xFFFFu) == my_target);
#pragma unroll
    for (int m = 0; m < N; ++m) ok = ok && (s.ent[m] & 0xFFFFu) != my_target;
    my_new = ok ? my_target : my_pos;
    // foods: lane `ag` decides foods ag, ag + N, ...
#pragma unroll
    for (int round = 0; round * N < F; ++round) {
      uint32_t fe = 0;  // level 0: nothing to decide
#pragma unroll
      for (int j = 0; j < N; ++j)
        if (round * N + j < F) fe = (ag == j) ? s.ent[N + round * N + j] : fe;
      const uint32_t fpos = fe & 0xFFFFu;
      const int fl = static_cast<int>(fe >> 16);
      int load = 0;
#pragma unroll
      for (int m = 0; m < N; ++m) {
        const uint32_t dist = __vsadu4(s.ent[m] & 0xFFFFu, fpos);  // |row difference| + |column difference|
        load += (((loaders >> m) & 1u) != 0u && dist == 1u) ? static_cast<int>(s.ent[m] >> 16) : 0;
      }
      const uint32_t bal = __ballot_sync(kFull, fl > 0 && load >= fl);
      collected_mask |= ((bal >> base) & ((1u << N) - 1u)) << (round * N);
    }
  } else {  // two agents: two shuffles are cheaper than a match across the warp
    // everybody's action and target, one shuffle per agent
    int act[N];
    uint32_t target[N];
    const uint32_t mine_packed = my_target | (static_cast<uint32_t>(action) << 16);
#pragma unroll
    for (int m = 0; m < N; ++m) {
      const uint32_t w = __shfl_sync(kFull, mine_packed, base + m);
      act[m] = static_cast<int>(w >> 16);
      target[m] = w & 0xFFFFu;
    }
    bool ok = my_target < 0xFFFEu;  // moving and inside the grid
#pragma unroll
    for (int f = 0; f < F; ++f) ok = ok && !((s.ent[N + f] >> 16) != 0 && (s.ent[N + f] & 0xFFFFu) == my_target);
#pragma unroll
    for (int m = 0; m < N; ++m)
      ok = ok && (m == ag || ((s.ent[m] & 0xFFFFu) != my_target && target[m] != my_target));
    my_new = ok ? my_target : my_pos;
    // foods: lane `ag` decides foods ag, ag + N, ...
#pragma unroll
    for (int round = 0; round * N < F; ++round) {
      uint32_t fe = 0;  // level 0: nothing to decide
#pragma unroll
      for (int j = 0; j < N; ++j)
        if (round * N + j < F) fe = (ag == j) ? s.ent[N + round * N + j] : fe;
      const int fr = fe & 0xFF, fc = (fe >> 8) & 0xFF, fl = static_cast<int>(fe >> 16);
      int load = 0;
#pragma unroll
      for (int m = 0; m < N; ++m) {
        const int dist = abs(static_cast<int>(s.ent[m] & 0xFF) - fr) + abs(static_cast<int>((s.ent[m] >> 8) & 0xFF) - fc);
        load += (act[m] == 5 && dist == 1) ? static_cast<int>(s.ent[m] >> 16) : 0;
      }
      const uint32_t bal = __ballot_sync(kFull, fl > 0 && load >= fl);
      collected_mask |= ((bal >> base) & ((1u << N) - 1u)) << (round * N);
    }
  }
  // apply: every lane updates its copy identically
  int gained = 0, left = 0;
#pragma unroll
  for (int m = 0; m < N; ++m) {
    const uint32_t np = __shfl_sync(kFull, my_new, base + m);
    s.ent[m] = (s.ent[m] & 0xFFFF0000u) | np;
  }
#pragma unroll
  for (int f = 0; f < F; ++f) {
    if ((collected_mask >> f) & 1u) { gained += static_cast<int>(s.ent[N + f] >> 16); s.ent[N + f] &= 0xFFFFu; }
    left += (s.ent[N + f] >> 16) != 0;
  }
  reward = gained > 0 ? __fdiv_rn(static_cast<float>(gained), static_cast<float>(s.total)) : 0.0f;
  s.step += 1;
  done = (left == 0) || (s.step >= p.cap);
  if (done && active) reset_env<N, F>(s, p, env, static_cast<uint32_t>(s.episode) + 1u);
}

}  // namespace mava
