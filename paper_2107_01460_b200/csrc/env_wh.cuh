// Device-side warehouse gridworld (the second workload family).  Same state containers as the foraging world:
// robot n = agent n with level 0 (empty-handed) or 1 + f (carrying shelf f); shelf f = "food" f with level 1 (idle) or
// 2 (requested), standing at its own cell or riding at its carrier's; EnvRec::total counts the episode's deliveries.
// Row 0 is the delivery row; floor(F/2) shelves (at least one) are requested at all times.
//
// Rules (every decision on the start-of-step state):
//   moves 1..4 are cancelled when the target is outside the grid, is another robot's current cell, is another mover's
//     target (those two are robot conflicts), or -- for a carrying robot -- holds a shelf that stands on the ground;
//   action 5 picks up the ground shelf the empty-handed robot stands under, or puts the carried shelf down unless the
//     robot is in the delivery row;
//   a carrying robot whose cell after the moves is in the delivery row delivers its shelf if that is requested: the
//     shelf turns idle, every robot is paid 1, and the d-th delivery of the step (robot order) draws a replacement
//     among the shelves that are idle and were not delivered in this step: word 0 of Philox(counter (d, env, episode,
//     step), request key) -> r in [0, n), the r-th such shelf in index order;
//   step += 1; done at the cap, or (env_kind 2) when a robot conflict cancelled a move.
// Two forms, as in env.cuh: on EnvRec records in shared memory (one thread per environment steps it), and on packed
// registers where every lane of an environment holds a full copy and applies identical integer updates.
#pragma once
#include "common.cuh"
#include "env.cuh"

namespace mava {

constexpr uint32_t kDomainRequest = 0x52455153u;  // key tweak of the replacement-request stream

__device__ __forceinline__ int wh_requests(int F) { return F / 2 > 0 ? F / 2 : 1; }

// ---- placement -------------------------------------------------------------------------------------------------------
// F shelf cells (r-th free cell of rows 1..G-1), N robot cells (r-th cell of the whole grid free of shelves and earlier
// robots), then the requests (r-th still idle shelf); draw i = word i % 4 of block (i / 4, env, episode, 0).
// cells[k]: shelves k = 0..F-1, then robots; status[f]: 1 or 2.
template <int N, int F>
__device__ void wh_place(const EnvParams &p, uint32_t env, uint32_t episode, int cells[N + F], int status[F]) {
  constexpr int K = N + F;
  constexpr int R = F / 2 > 0 ? F / 2 : 1;
  constexpr int NBLK = (K + R + 3) / 4;
  uint32_t draws[NBLK * 4];
#pragma unroll
  for (int b = 0; b < NBLK; ++b)
    philox4x32_10(static_cast<uint32_t>(b), env, episode, 0u, p.key_lo, p.key_hi ^ kDomainReset, &draws[4 * b]);
  const int G = p.grid;
  int taken[K];  // sorted cells taken so far
#pragma unroll
  for (int k = 0; k < K; ++k) {
    const int first = k < F ? G : 0;  // shelves start at row 1
    const int n_free = (k < F ? (G - 1) * G : G * G) - k;
    int cell = first + static_cast<int>(bounded(draws[k], static_cast<uint32_t>(n_free)));
#pragma unroll
    for (int j = 0; j < K; ++j)
      if (j < k && taken[j] <= cell) ++cell;  // all taken cells so far lie at or after `first` for shelves; robots count all
    cells[k] = cell;
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
#pragma unroll
  for (int f = 0; f < F; ++f) status[f] = 1;
#pragma unroll
  for (int k = 0; k < R; ++k) {
    int r = static_cast<int>(bounded(draws[K + k], static_cast<uint32_t>(F - k)));
#pragma unroll
    for (int f = 0; f < F; ++f) {
      if (status[f] == 1) {
        if (r == 0) status[f] = 2;
        --r;
      }
    }
  }
}

// ---- EnvRec form ---------------------------------------------------------------------------------------------------------
template <int N, int F>
__device__ void wh_reset_rec(EnvRec &s, const EnvParams &p, uint32_t env, uint32_t episode) {
  int cells[N + F], status[F];
  wh_place<N, F>(p, env, episode, cells, status);
  const int G = p.grid;
#pragma unroll
  for (int f = 0; f < F; ++f) {
    s.fr[f] = static_cast<uint8_t>(cells[f] / G); s.fc[f] = static_cast<uint8_t>(cells[f] % G); s.fl[f] = static_cast<uint8_t>(status[f]);
  }
#pragma unroll
  for (int n = 0; n < N; ++n) {
    s.ar[n] = static_cast<uint8_t>(cells[F + n] / G); s.ac[n] = static_cast<uint8_t>(cells[F + n] % G); s.al[n] = 0;
  }
  s.step = 0; s.episode = static_cast<int32_t>(episode); s.total = 0;
}

// Element j of the observation of robot `a` (dense form, for the fp32 path).
template <int N, int F>
__device__ __forceinline__ float wh_obs_element(const EnvRec &s, const EnvParams &p, int a, int j) {
  const int G = p.grid;
  if (j < 3 * kPlane) {
    const int plane = j / kPlane, q = j - plane * kPlane;
    const int rr = static_cast<int>(s.ar[a]) + q / kWindow - kViewRadius, cc = static_cast<int>(s.ac[a]) + q % kWindow - kViewRadius;
    const bool outside = rr < 0 || rr >= G || cc < 0 || cc >= G;
    if (plane == 2) return outside ? 1.0f : (rr == 0 ? 0.5f : 0.0f);
    if (outside) return 0.0f;
    float v = 0.0f;
    if (plane == 0) {
#pragma unroll
      for (int n = 0; n < N; ++n)
        if (s.ar[n] == rr && s.ac[n] == cc) v = s.al[n] > 0 ? 2.0f : 1.0f;
    } else {
#pragma unroll
      for (int f = 0; f < F; ++f)
        if (s.fr[f] == rr && s.fc[f] == cc) v = static_cast<float>(s.fl[f]);
    }
    return v;
  }
  if (j == 3 * kPlane) return s.al[a] > 0 ? 2.0f : 1.0f;
  if (j == 3 * kPlane + 1) return __fdiv_rn(static_cast<float>(s.step), static_cast<float>(p.cap));
  return (j - kObsFixed == a) ? 1.0f : 0.0f;
}

// The whole transition of one environment on plain arrays: pos[k] = row | col << 8 (robots 0..N-1, then shelves),
// carry[n], status[f].  Returns the number of deliveries; `conflict` reports a robot conflict.
template <int N, int F>
__device__ __forceinline__ int wh_transition(uint32_t pos[N + F], int carry[N], int status[F], const int act[N], const EnvParams &p,
                                             uint32_t env, uint32_t episode, uint32_t step, bool &conflict) {
  const int G = p.grid;
  uint32_t target[N];
  bool ok[N];
  uint32_t on_robot = 0;  // bit f: shelf f rides on a robot at the start of the step
#pragma unroll
  for (int n = 0; n < N; ++n) on_robot |= carry[n] > 0 ? 1u << (carry[n] - 1) : 0u;
#pragma unroll
  for (int n = 0; n < N; ++n) {
    const int r = pos[n] & 0xFF, c = pos[n] >> 8, a = act[n];
    const int tr = r + (a == 2) - (a == 1), tc = c + (a == 4) - (a == 3);
    const bool moving = a >= 1 && a <= 4, inside = tr >= 0 && tr < G && tc >= 0 && tc < G;
    target[n] = moving ? (inside ? (static_cast<uint32_t>(tr) | (static_cast<uint32_t>(tc) << 8)) : 0xFFFEu) : 0xFFFFu;
  }
  conflict = false;
#pragma unroll
  for (int n = 0; n < N; ++n) {
    ok[n] = target[n] < 0xFFFEu;
    if (target[n] != 0xFFFFu) {  // a mover, also one headed off the grid: conflicts are judged on its target cell
      bool clash = false;
#pragma unroll
      for (int m = 0; m < N; ++m)
        if (m != n) clash = clash || (target[n] < 0xFFFEu && (pos[m] == target[n] || target[m] == target[n]));
      conflict = conflict || clash;
      ok[n] = ok[n] && !clash;
      if (carry[n] > 0) {
#pragma unroll
        for (int f = 0; f < F; ++f) ok[n] = ok[n] && !(((on_robot >> f) & 1u) == 0 && pos[N + f] == target[n]);
      }
    }
  }
  int new_carry[N];
#pragma unroll
  for (int n = 0; n < N; ++n) {
    new_carry[n] = carry[n];
    if (act[n] == 5) {
      if (carry[n] == 0) {
#pragma unroll
        for (int f = 0; f < F; ++f)
          if (((on_robot >> f) & 1u) == 0 && pos[N + f] == pos[n]) new_carry[n] = 1 + f;
      } else if ((pos[n] & 0xFF) != 0) {
        new_carry[n] = 0;
      }
    }
  }
#pragma unroll
  for (int n = 0; n < N; ++n) {
    carry[n] = new_carry[n];
    if (ok[n]) {
      pos[n] = target[n];
#pragma unroll
      for (int f = 0; f < F; ++f)
        if (carry[n] == 1 + f) pos[N + f] = target[n];
    }
  }
  uint32_t delivered = 0;
  int d = 0;
#pragma unroll
  for (int n = 0; n < N; ++n) {
#pragma unroll
    for (int f = 0; f < F; ++f)
      if (carry[n] == 1 + f && (pos[n] & 0xFF) == 0 && status[f] == 2) { status[f] = 1; delivered |= 1u << f; ++d; }
  }
  for (int k = 0; k < d; ++k) {
    int n_idle = 0;
#pragma unroll
    for (int f = 0; f < F; ++f) n_idle += (status[f] == 1 && ((delivered >> f) & 1u) == 0);
    if (n_idle == 0) break;
    uint32_t o[4];
    philox4x32_10(static_cast<uint32_t>(k), env, episode, step, p.key_lo, p.key_hi ^ kDomainRequest, o);
    int r = static_cast<int>(bounded(o[0], static_cast<uint32_t>(n_idle)));
#pragma unroll
    for (int f = 0; f < F; ++f) {
      if (status[f] == 1 && ((delivered >> f) & 1u) == 0) {
        if (r == 0) status[f] = 2;
        --r;
      }
    }
  }
  return d;
}

// One thread steps the environment `s` with the actions act[0..N); starts the next episode when done.
template <int N, int F>
__device__ __forceinline__ void wh_step_rec(EnvRec &s, const EnvParams &p, uint32_t env, const int *act_in, float &reward, bool &done) {
  uint32_t pos[N + F];
  int carry[N], status[F], act[N];
#pragma unroll
  for (int n = 0; n < N; ++n) { pos[n] = s.ar[n] | (static_cast<uint32_t>(s.ac[n]) << 8); carry[n] = s.al[n]; act[n] = act_in[n]; }
#pragma unroll
  for (int f = 0; f < F; ++f) { pos[N + f] = s.fr[f] | (static_cast<uint32_t>(s.fc[f]) << 8); status[f] = s.fl[f]; }
  bool conflict;
  const int d = wh_transition<N, F>(pos, carry, status, act, p, env, static_cast<uint32_t>(s.episode), static_cast<uint32_t>(s.step), conflict);
#pragma unroll
  for (int n = 0; n < N; ++n) { s.ar[n] = static_cast<uint8_t>(pos[n]); s.ac[n] = static_cast<uint8_t>(pos[n] >> 8); s.al[n] = static_cast<uint8_t>(carry[n]); }
#pragma unroll
  for (int f = 0; f < F; ++f) { s.fr[f] = static_cast<uint8_t>(pos[N + f]); s.fc[f] = static_cast<uint8_t>(pos[N + f] >> 8); s.fl[f] = static_cast<uint8_t>(status[f]); }
  s.total += d;
  reward = static_cast<float>(d);
  s.step += 1;
  done = (s.step >= p.cap) || (p.env_kind == 2 && conflict);
  if (done) wh_reset_rec<N, F>(s, p, env, static_cast<uint32_t>(s.episode) + 1u);
}

// ---- register form -----------------------------------------------------------------------------------------------------
template <int N, int F>
__device__ void wh_reset_env(EnvRegs<N, F> &s, const EnvParams &p, uint32_t env, uint32_t episode) {
  int cells[N + F], status[F];
  wh_place<N, F>(p, env, episode, cells, status);
  const int G = p.grid;
#pragma unroll
  for (int n = 0; n < N; ++n) s.ent[n] = pack_entity(cells[F + n] / G, cells[F + n] % G, 0);
#pragma unroll
  for (int f = 0; f < F; ++f) s.ent[N + f] = pack_entity(cells[f] / G, cells[f] % G, status[f]);
  s.step = 0; s.episode = static_cast<int32_t>(episode); s.total = 0;
}

// Non-zero observation entries of robot `ag`.
template <int N, int F, class Sink>
__device__ __forceinline__ void wh_observe_env(const EnvRegs<N, F> &s, const EnvParams &p, int ag, Sink sink) {
  const uint32_t me = own_entity(s, ag);
  const int r0 = me & 0xFF, c0 = (me >> 8) & 0xFF, G = p.grid;
#pragma unroll
  for (int dy = 0; dy < kWindow; ++dy) {
    const int rr = r0 + dy - kViewRadius;
#pragma unroll
    for (int dx = 0; dx < kWindow; ++dx) {
      const int cc = c0 + dx - kViewRadius;
      const bool outside = rr < 0 || rr >= G || cc < 0 || cc >= G;
      if (outside) sink(2 * kPlane + dy * kWindow + dx, 1.0f);
      else if (rr == 0) sink(2 * kPlane + dy * kWindow + dx, 0.5f);
    }
  }
#pragma unroll
  for (int k = 0; k < N + F; ++k) {
    const uint32_t e = s.ent[k];
    const int dy = static_cast<int>(e & 0xFF) - r0 + kViewRadius, dx = static_cast<int>((e >> 8) & 0xFF) - c0 + kViewRadius;
    const int lvl = static_cast<int>(e >> 16);
    if (dy >= 0 && dy < kWindow && dx >= 0 && dx < kWindow) {
      if (k < N) sink(dy * kWindow + dx, lvl > 0 ? 2.0f : 1.0f);
      else sink(kPlane + dy * kWindow + dx, static_cast<float>(lvl));
    }
  }
  sink(3 * kPlane, (me >> 16) != 0 ? 2.0f : 1.0f);
  sink(3 * kPlane + 1, __fdiv_rn(static_cast<float>(s.step), static_cast<float>(p.cap)));
  sink(kObsFixed + ag, 1.0f);
}

// One transition of the environment whose N robot threads occupy lanes [base, base + N): every lane of the warp
// calls it; the lanes of an environment exchange their actions and then each applies the whole transition to its
// own copy of the state, so the copies stay identical.
template <int N, int F>
__device__ __forceinline__ void wh_step_env_warp(EnvRegs<N, F> &s, const EnvParams &p, uint32_t env, int base, bool active, int action,
                                                 float &reward, bool &done) {
  int act[N];
#pragma unroll
  for (int m = 0; m < N; ++m) act[m] = __shfl_sync(0xFFFFFFFFu, action, base + m);
  uint32_t pos[N + F];
  int carry[N], status[F];
#pragma unroll
  for (int n = 0; n < N; ++n) { pos[n] = s.ent[n] & 0xFFFFu; carry[n] = static_cast<int>(s.ent[n] >> 16); }
#pragma unroll
  for (int f = 0; f < F; ++f) { pos[N + f] = s.ent[N + f] & 0xFFFFu; status[f] = static_cast<int>(s.ent[N + f] >> 16); }
  bool conflict;
  const int d = wh_transition<N, F>(pos, carry, status, act, p, env, static_cast<uint32_t>(s.episode), static_cast<uint32_t>(s.step), conflict);
#pragma unroll
  for (int n = 0; n < N; ++n) s.ent[n] = pos[n] | (static_cast<uint32_t>(carry[n]) << 16);
#pragma unroll
  for (int f = 0; f < F; ++f) s.ent[N + f] = pos[N + f] | (static_cast<uint32_t>(status[f]) << 16);
  s.total += d;
  reward = static_cast<float>(d);
  s.step += 1;
  done = (s.step >= p.cap) || (p.env_kind == 2 && conflict);
  if (done && active) wh_reset_env<N, F>(s, p, env, static_cast<uint32_t>(s.episode) + 1u);
}

}  // namespace mava
