// Host-side offsets of the dense layers inside a flat parameter array.
#pragma once
#include <stddef.h>

#include "mava_rollout.h"

namespace mava {

struct ParamLayout {
  size_t W1, b1, W2, b2, Wa, ba, Wv, bv;  // Wv/bv unused with the central critic
  size_t C1, c1, C2, c2, Cv, cv;          // central critic only
  size_t Wih, bih, Whh, bhh;              // recurrent policy only: the cell's matrices [3H][H] and biases [3H] (gates r, z, n)
  size_t total;
};

// `align` = 1 gives the caller-facing layout; a larger value rounds every segment start up to a
// multiple of `align` floats (library-internal copies that are read with vector loads).
inline ParamLayout param_layout(const mava_config_t &cfg, int D, size_t align) {
  ParamLayout L{};
  const size_t H = static_cast<size_t>(cfg.hidden), N = static_cast<size_t>(cfg.n_agents);
  size_t off = 0;
  auto take = [&](size_t n) {
    off = (off + align - 1) / align * align;
    const size_t at = off;
    off += n;
    return at;
  };
  L.W1 = take(H * D); L.b1 = take(H);
  if (cfg.net_kind == MAVA_NET_RECURRENT) {
    L.Wih = take(3 * H * H); L.bih = take(3 * H);
    L.Whh = take(3 * H * H); L.bhh = take(3 * H);
    L.Wa = take(MAVA_N_ACTIONS * H); L.ba = take(MAVA_N_ACTIONS);
    L.Wv = take(H); L.bv = take(1);
    L.total = (off + align - 1) / align * align;
    return L;
  }
  L.W2 = take(H * H); L.b2 = take(H);
  L.Wa = take(MAVA_N_ACTIONS * H); L.ba = take(MAVA_N_ACTIONS);
  if (cfg.net_kind == MAVA_NET_SHARED_TORSO) {
    L.Wv = take(H); L.bv = take(1);
  } else {
    L.C1 = take(H * N * D); L.c1 = take(H);
    L.C2 = take(H * H); L.c2 = take(H);
    L.Cv = take(H); L.cv = take(1);
  }
  L.total = (off + align - 1) / align * align;
  return L;
}

}  // namespace mava
