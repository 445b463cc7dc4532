// Update block, first correct path (fp32 on the plain ALUs): the multi-agent PPO loss of one minibatch (all rows
// of the last rollout), its gradient with respect to every parameter, and the Adam step.
//   loss:  rho = exp(logp_new(a) - logp_old);  Ahat = (A - mean A) / (std A + 1e-8);
//          L = -mean min(rho Ahat, clip(rho, 1 +- eps) Ahat) - c_ent mean H
//              + c_val 0.5 mean max((V - R)^2, (Vold + clip(V - Vold, +-eps) - R)^2)
// A CTA of H threads (thread j = hidden unit j) walks over tiles of 32 rows: forward through the two hidden
// layers with the activations of the tile in shared memory, heads and per-row loss derivatives by one warp per
// row, backward through the layers, and the tile's contribution to every weight gradient added into the CTA's
// own slice of a partial-gradient array (reductions without a return value: an address is only ever added to by
// one thread, in program order; a last kernel adds the slices in a fixed order, so the result does not depend
// on scheduling).  Sums that decide a mean are kept in double.
// This is the validation path of the update block, as rollout_simt.cu is the rollout's; a tensor-core path
// (the weight gradients are GEMMs over millions of rows) is not built yet.
#include "common.cuh"
#include "layout.h"
#include "update_common.cuh"

namespace mava {
namespace {

constexpr int kUpdRows = 32;       // rows per tile
constexpr int kUpdTS = kUpdRows;   // row stride of the transposed d z tiles [unit][row] (read by 16-byte broadcasts; the few
                                   // stores that fill them collide on banks, which costs less than the room padding takes)
constexpr int kStatBlocks = 256;   // partial sums of the two reductions

__global__ void transpose_kernel(const float *__restrict__ W, float *__restrict__ Wt, int out, int in) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < out * in; i += gridDim.x * blockDim.x) {
    const int o = i / in, k = i - o * in;
    Wt[static_cast<size_t>(k) * out + o] = W[i];
  }
}

// Block partial sums of x and x^2 (double), then one block turns them into mean and population std.
__global__ void stat_partial_kernel(const float *__restrict__ x, long long n, double *__restrict__ part, UpdRows map) {
  __shared__ double s0[256], s1[256];
  double a = 0.0, b = 0.0;
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += static_cast<long long>(gridDim.x) * blockDim.x) {
    const long long row = real_row(map, i);
    const double v = row >= 0 ? x[row] : 0.0;
    a += v; b += v * v;
  }
  s0[threadIdx.x] = a; s1[threadIdx.x] = b;
  __syncthreads();
  for (int k = blockDim.x / 2; k > 0; k /= 2) {
    if (threadIdx.x < k) { s0[threadIdx.x] += s0[threadIdx.x + k]; s1[threadIdx.x] += s1[threadIdx.x + k]; }
    __syncthreads();
  }
  if (threadIdx.x == 0) { part[2 * blockIdx.x] = s0[0]; part[2 * blockIdx.x + 1] = s1[0]; }
}
// One warp; lane l adds its contiguous share of the partials, lane 0 the 32 shares: the same order on every call.
__global__ void stat_final_kernel(const double *__restrict__ part, int nb, long long n, double *__restrict__ out) {
  __shared__ double sa[32], sb[32];
  const int per = (nb + 31) / 32, lane = threadIdx.x;
  double a = 0.0, b = 0.0;
  for (int i = lane * per; i < min(nb, (lane + 1) * per); ++i) { a += part[2 * i]; b += part[2 * i + 1]; }
  sa[lane] = a; sb[lane] = b;
  __syncwarp();
  if (lane != 0) return;
  a = 0.0; b = 0.0;
  for (int i = 0; i < 32; ++i) { a += sa[i]; b += sb[i]; }
  const double mean = a / static_cast<double>(n);
  const double var = fmax(b / static_cast<double>(n) - mean * mean, 0.0);
  out[0] = mean; out[1] = sqrt(var); out[2] = sqrt(b);  // [2]: the 2-norm, for the gradient clipping
}


// HT = hidden width = threads per CTA; the register budget is set for the CTAs per SM that the shared memory allows.
template <int HT>
__global__ void __launch_bounds__(HT, HT == 256 ? 1 : (HT == 128 ? 3 : 4))
ppo_net_kernel(UpdNet net, UpdRows rows, UpdHyper hp, const double *__restrict__ adv_stats,
                               float *__restrict__ partial, size_t n_params, double *__restrict__ term_partial, int *status) {
  extern __shared__ __align__(16) float smf[];
  constexpr int H = HT;
  const int Din = net.Din, j = threadIdx.x, lane = j & 31, warp = j >> 5, n_warps = H >> 5;
  const int Dp = (Din + 3) & ~3;  // row stride of the input tile; the pad columns hold zeros
  // every inner product below reads four operands per shared-memory access (16-byte broadcast loads)
  // d z1 takes the place of h2, which is dead by then: three CTAs fit an SM at H = 128
  float *xs = smf, *h1s = xs + kUpdRows * Dp, *h2s = h1s + kUpdRows * H, *dz2t = h2s + kUpdRows * H, *dz1t = h2s,
        *dl = dz2t + H * kUpdTS;  // dl [32][8]: d logits (6), d value
  long long *rmap = reinterpret_cast<long long *>(dl + kUpdRows * 8);  // trajectory row of every row of the tile
  auto ld4 = [](const float *p) { return *reinterpret_cast<const float4 *>(p); };
  const int HH = H >> 1, up = j % HH, r0 = (j / HH) * (kUpdRows / 2);  // the two-unit mapping of the dense loops
  float *part = partial + static_cast<size_t>(blockIdx.x) * n_params;
  const bool has_actor = net.Wa != nullptr, has_value = net.Wv != nullptr;
  const float mean = has_actor ? static_cast<float>(adv_stats[0]) : 0.0f;
  const float inv_std = has_actor ? 1.0f / (static_cast<float>(adv_stats[1]) + 1e-8f) : 0.0f;
  const float inv_n = 1.0f / static_cast<float>(rows.n);
  float gWa[kActions], gWv = 0.0f, gb1 = 0.0f, gb2 = 0.0f, gbh = 0.0f;
#pragma unroll
  for (int k = 0; k < kActions; ++k) gWa[k] = 0.0f;
  double t_actor = 0.0, t_ent = 0.0, t_value = 0.0;  // lane 0 of every warp
  const long long n_tiles = (rows.n + kUpdRows - 1) / kUpdRows;
  for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const long long row0 = tile * kUpdRows;
    const int n_valid = static_cast<int>(min(static_cast<long long>(kUpdRows), rows.n - row0));
    if (j < kUpdRows) {
      const long long row = j < n_valid ? real_row(rows, row0 + j) : -1;
      rmap[j] = row;
      if (j < n_valid && row < 0) atomicExch(status, kStatusBadIndex);
    }
    __syncthreads();
    for (int r = warp; r < kUpdRows; r += n_warps) {  // a warp per row: consecutive lanes, consecutive floats
      const long long row = rmap[r];
      for (int k = lane; k < Dp; k += 32) xs[r * Dp + k] = (row >= 0 && k < Din) ? rows.x[row * Din + k] : 0.0f;
    }
    __syncthreads();
    // hidden layer 1 and 2.  Here a thread computes two units (up, up + H/2) of half the tile's rows, so that one
    // 16-byte broadcast read of the activations feeds eight multiply-adds.
    auto dense2 = [&](const float *src, int stride, int K, int k_valid, const float *Wt, const float *bias, float *dst) {
      float a0[kUpdRows / 2], a1[kUpdRows / 2];
#pragma unroll
      for (int r = 0; r < kUpdRows / 2; ++r) a0[r] = a1[r] = 0.0f;
      for (int k = 0; k < K; k += 4) {
        float w0[4], w1[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const bool ok = k + q < k_valid;
          w0[q] = ok ? Wt[static_cast<size_t>(k + q) * H + up] : 0.0f;
          w1[q] = ok ? Wt[static_cast<size_t>(k + q) * H + up + HH] : 0.0f;
        }
#pragma unroll
        for (int r = 0; r < kUpdRows / 2; ++r) {
          const float4 x = ld4(src + (r0 + r) * stride + k);
          a0[r] = fmaf(x.x, w0[0], fmaf(x.y, w0[1], fmaf(x.z, w0[2], fmaf(x.w, w0[3], a0[r]))));
          a1[r] = fmaf(x.x, w1[0], fmaf(x.y, w1[1], fmaf(x.z, w1[2], fmaf(x.w, w1[3], a1[r]))));
        }
      }
      const float b0 = bias[up], b1v = bias[up + HH];
#pragma unroll
      for (int r = 0; r < kUpdRows / 2; ++r) {
        dst[(r0 + r) * H + up] = fmaxf(a0[r] + b0, 0.0f);
        dst[(r0 + r) * H + up + HH] = fmaxf(a1[r] + b1v, 0.0f);
      }
    };
    dense2(xs, Dp, Dp, Din, net.W1t, net.b1, h1s);
    __syncthreads();
    dense2(h1s, H, H, H, net.W2t, net.b2, h2s);
    __syncthreads();
    // heads and the per-row derivatives of the loss: one warp per row
    for (int r = warp; r < kUpdRows; r += n_warps) {
      float s[kActions + 1];
#pragma unroll
      for (int k = 0; k <= kActions; ++k) s[k] = 0.0f;
      for (int i = lane; i < H; i += 32) {
        const float hv = h2s[r * H + i];
        if (has_actor) {
#pragma unroll
          for (int k = 0; k < kActions; ++k) s[k] = fmaf(hv, net.Wa[k * H + i], s[k]);
        }
        if (has_value) s[kActions] = fmaf(hv, net.Wv[i], s[kActions]);
      }
#pragma unroll
      for (int k = 0; k <= kActions; ++k)
        for (int o = 16; o > 0; o >>= 1) s[k] += __shfl_xor_sync(0xFFFFFFFFu, s[k], o);
      if (lane == 0) {
        float d[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) d[k] = 0.0f;
        if (rmap[r] >= 0) {
          const long long row = rmap[r];
          if (has_actor) {
            float l[kActions], m = -INFINITY, sum = 0.0f;
#pragma unroll
            for (int k = 0; k < kActions; ++k) { l[k] = s[k] + net.ba[k]; m = fmaxf(m, l[k]); }
#pragma unroll
            for (int k = 0; k < kActions; ++k) sum += expf(l[k] - m);
            const float lse = m + logf(sum);
            const int a = rows.actions[row];
            float ent = 0.0f, p[kActions], lp[kActions], lpa = 0.0f;
#pragma unroll
            for (int k = 0; k < kActions; ++k) {
              lp[k] = l[k] - lse; p[k] = expf(lp[k]); ent -= p[k] * lp[k];
              if (k == a) lpa = lp[k];
            }
            const float rho = expf(lpa - rows.logp_old[row]);
            const float ahat = (rows.adv[row] - mean) * inv_std;
            const float clipped = fminf(fmaxf(rho, 1.0f - hp.clip_eps), 1.0f + hp.clip_eps);
            const float s1 = rho * ahat, s2 = clipped * ahat;
            const bool inside = rho >= 1.0f - hp.clip_eps && rho <= 1.0f + hp.clip_eps;
            const float d_logp = (inside || s1 < s2) ? -s1 * inv_n : 0.0f;  // the clipped branch is constant in rho
#pragma unroll
            for (int k = 0; k < kActions; ++k)
              d[k] = d_logp * ((k == a ? 1.0f : 0.0f) - p[k]) + hp.ent_coef * inv_n * p[k] * (lp[k] + ent);
            t_actor += fminf(s1, s2);
            t_ent += ent;
          }
          if (has_value) {
            const float v = s[kActions] + net.bv[0], vo = rows.value_old[row * rows.vstride], rt = rows.ret[row * rows.vstride];
            const float u = v - rt, uc = vo + fminf(fmaxf(v - vo, -hp.clip_eps), hp.clip_eps) - rt;
            const bool in_range = fabsf(v - vo) <= hp.clip_eps;
            d[kActions] = (in_range || u * u > uc * uc) ? hp.vf_coef * u * inv_n : 0.0f;
            t_value += 0.5 * fmaxf(u * u, uc * uc);
          }
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) dl[r * 8 + k] = d[k];
      }
    }
    __syncthreads();
    // back through the heads: d h2, head gradients (kept in registers over all tiles), d z2
    float dzr[kUpdRows];
#pragma unroll
    for (int r = 0; r < kUpdRows; ++r) {
      const float hv = h2s[r * H + j];
      float dh = 0.0f;
      if (has_actor) {
#pragma unroll
        for (int k = 0; k < kActions; ++k) {
          const float dk = dl[r * 8 + k];
          dh = fmaf(dk, net.Wa[k * H + j], dh);
          gWa[k] = fmaf(dk, hv, gWa[k]);
        }
      }
      if (has_value) {
        const float dv = dl[r * 8 + kActions];
        dh = fmaf(dv, net.Wv[j], dh);
        gWv = fmaf(dv, hv, gWv);
      }
      const float dz = hv > 0.0f ? dh : 0.0f;
      dzr[r] = dz;
      gb2 += dz;
      if (j < 8) gbh += dl[r * 8 + j];  // threads 0..6: the heads' biases
    }
#pragma unroll
    for (int r = 0; r < kUpdRows; r += 4)
      *reinterpret_cast<float4 *>(dz2t + j * kUpdTS + r) = make_float4(dzr[r], dzr[r + 1], dzr[r + 2], dzr[r + 3]);
    __syncthreads();
    // d h1 = d z2 . W2 (rows of W2 are contiguous in the unit index), d z1: again two units and half the rows per thread
    {
      float a0[kUpdRows / 2], a1[kUpdRows / 2];
#pragma unroll
      for (int r = 0; r < kUpdRows / 2; ++r) a0[r] = a1[r] = 0.0f;
      for (int i = 0; i < H; i += 4) {
        float w0[4], w1[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          w0[q] = net.W2[static_cast<size_t>(i + q) * H + up];
          w1[q] = net.W2[static_cast<size_t>(i + q) * H + up + HH];
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
#pragma unroll
          for (int r = 0; r < kUpdRows / 2; r += 4) {
            const float4 d = ld4(dz2t + (i + q) * kUpdTS + r0 + r);
            a0[r] = fmaf(d.x, w0[q], a0[r]); a0[r + 1] = fmaf(d.y, w0[q], a0[r + 1]);
            a0[r + 2] = fmaf(d.z, w0[q], a0[r + 2]); a0[r + 3] = fmaf(d.w, w0[q], a0[r + 3]);
            a1[r] = fmaf(d.x, w1[q], a1[r]); a1[r + 1] = fmaf(d.y, w1[q], a1[r + 1]);
            a1[r + 2] = fmaf(d.z, w1[q], a1[r + 2]); a1[r + 3] = fmaf(d.w, w1[q], a1[r + 3]);
          }
        }
      }
      // d z1 takes h2's place: h2 was last read before the barrier that precedes this loop
#pragma unroll
      for (int r = 0; r < kUpdRows / 2; r += 4) {
        float4 z0, z1;
        z0.x = h1s[(r0 + r) * H + up] > 0.0f ? a0[r] : 0.0f; z0.y = h1s[(r0 + r + 1) * H + up] > 0.0f ? a0[r + 1] : 0.0f;
        z0.z = h1s[(r0 + r + 2) * H + up] > 0.0f ? a0[r + 2] : 0.0f; z0.w = h1s[(r0 + r + 3) * H + up] > 0.0f ? a0[r + 3] : 0.0f;
        z1.x = h1s[(r0 + r) * H + up + HH] > 0.0f ? a1[r] : 0.0f; z1.y = h1s[(r0 + r + 1) * H + up + HH] > 0.0f ? a1[r + 1] : 0.0f;
        z1.z = h1s[(r0 + r + 2) * H + up + HH] > 0.0f ? a1[r + 2] : 0.0f; z1.w = h1s[(r0 + r + 3) * H + up + HH] > 0.0f ? a1[r + 3] : 0.0f;
        *reinterpret_cast<float4 *>(dz1t + up * kUpdTS + r0 + r) = z0;
        *reinterpret_cast<float4 *>(dz1t + (up + HH) * kUpdTS + r0 + r) = z1;
      }
    }
    __syncthreads();
    // bias gradient of layer 1: thread j sums d z1 of unit j over the tile's rows
#pragma unroll
    for (int r = 0; r < kUpdRows; r += 4) {
      const float4 d = ld4(dz1t + j * kUpdTS + r);
      gb1 += (d.x + d.y) + (d.z + d.w);
    }
    // Weight gradients, G[i][c] += sum_r dz[r][i] v[r][c]: a thread keeps two columns c of v (all 32 rows) in registers
    // and walks over half of the units i, so that every address is added to by one thread only and a broadcast read of
    // d z feeds eight multiply-adds.
    auto weight_grad = [&](const float *dzt, const float *v, int v_stride, int n_cols, size_t g_off) {
      const int i0 = (j / HH) * HH;
      for (int cb = 0; cb < n_cols; cb += H) {
        const int c0 = cb + up, c1 = cb + up + HH;
        if (c0 >= n_cols) break;
        const bool two = c1 < n_cols;
        float v0[kUpdRows], v1[kUpdRows];
#pragma unroll
        for (int r = 0; r < kUpdRows; ++r) {
          v0[r] = v[r * v_stride + c0];
          v1[r] = two ? v[r * v_stride + c1] : 0.0f;
        }
        for (int i = i0; i < i0 + HH; ++i) {
          float s0 = 0.0f, s1 = 0.0f;
#pragma unroll
          for (int r = 0; r < kUpdRows; r += 4) {
            const float4 d = ld4(dzt + i * kUpdTS + r);
            s0 = fmaf(d.x, v0[r], fmaf(d.y, v0[r + 1], fmaf(d.z, v0[r + 2], fmaf(d.w, v0[r + 3], s0))));
            s1 = fmaf(d.x, v1[r], fmaf(d.y, v1[r + 1], fmaf(d.z, v1[r + 2], fmaf(d.w, v1[r + 3], s1))));
          }
          // results unused: fire-and-forget reductions, no load to wait for
          atomicAdd(part + g_off + static_cast<size_t>(i) * n_cols + c0, s0);
          if (two) atomicAdd(part + g_off + static_cast<size_t>(i) * n_cols + c1, s1);
        }
      }
    };
    weight_grad(dz2t, h1s, H, H, net.oW2);    // d W2[i][j] = sum_r d z2[r][i] h1[r][j]
    weight_grad(dz1t, xs, Dp, Din, net.oW1);  // d W1[i][k] = sum_r d z1[r][i] x[r][k]
    __syncthreads();
  }
  // what was kept in registers over all tiles
  part[net.ob1 + j] += gb1;
  part[net.ob2 + j] += gb2;
  if (has_actor) {
#pragma unroll
    for (int k = 0; k < kActions; ++k) part[net.oWa + static_cast<size_t>(k) * H + j] += gWa[k];
    if (j < kActions) part[net.oba + j] += gbh;
  }
  if (has_value) {
    part[net.oWv + j] += gWv;
    if (j == kActions) part[net.obv] += gbh;
  }
  if (lane == 0) {
    double *tp = term_partial + (static_cast<size_t>(blockIdx.x) * 8 + warp) * 3;
    tp[0] += t_actor; tp[1] += t_ent; tp[2] += t_value;
  }
}

// grad[p] = sum over the CTAs' slices, in slice order; block 0 also turns the term sums into the loss terms.
__global__ void reduce_partials_kernel(const float *__restrict__ partial, size_t n_params, int n_slices, float *__restrict__ grad,
                                       const double *__restrict__ term_partial, int n_term, long long n_actor, long long n_value,
                                       UpdHyper hp, float *__restrict__ terms) {
  for (size_t p = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; p < n_params; p += static_cast<size_t>(gridDim.x) * blockDim.x) {
    float s = 0.0f;
#pragma unroll 8
    for (int c = 0; c < n_slices; ++c) s += partial[static_cast<size_t>(c) * n_params + p];  // the loads do not wait for the sum
    grad[p] = s;
  }
  if (blockIdx.x != 0 || !terms) return;
  // the loss terms: every thread of block 0 adds a contiguous share of the partial sums, thread 0 the shares
  __shared__ double st[3][256];
  {
    const int per = (n_term + static_cast<int>(blockDim.x) - 1) / static_cast<int>(blockDim.x), t = threadIdx.x;
    double a = 0.0, e = 0.0, v = 0.0;
    for (int i = t * per; i < min(n_term, (t + 1) * per); ++i) { a += term_partial[3 * i]; e += term_partial[3 * i + 1]; v += term_partial[3 * i + 2]; }
    st[0][t] = a; st[1][t] = e; st[2][t] = v;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double a = 0.0, e = 0.0, v = 0.0;
    for (int i = 0; i < static_cast<int>(blockDim.x); ++i) { a += st[0][i]; e += st[1][i]; v += st[2][i]; }
    const double actor = -a / static_cast<double>(n_actor), ent = e / static_cast<double>(n_actor), val = v / static_cast<double>(n_value);
    terms[0] = static_cast<float>(actor - hp.ent_coef * ent + hp.vf_coef * val);
    terms[1] = static_cast<float>(actor);
    terms[2] = static_cast<float>(ent);
    terms[3] = static_cast<float>(val);
  }
}

__global__ void adam_kernel(float *__restrict__ params, const float *__restrict__ grad, float *__restrict__ m, float *__restrict__ v,
                            size_t n, const double *__restrict__ stats, float max_norm, float lr, float beta1, float beta2,
                            float eps, float corr1, float corr2) {
  const float norm = static_cast<float>(stats[2]);
  const float scale = max_norm / fmaxf(norm, max_norm);
  for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += static_cast<size_t>(gridDim.x) * blockDim.x) {
    const float g = grad[i] * scale;
    const float mi = beta1 * m[i] + (1.0f - beta1) * g, vi = beta2 * v[i] + (1.0f - beta2) * g * g;
    m[i] = mi; v[i] = vi;
    params[i] -= lr * (mi / corr1) / (sqrtf(vi / corr2) + eps);
  }
}

// Scratch of the update block, made on first use: [stats: 3 doubles][stat partials][term partials][transposed
// weights][partial gradients: one slice per CTA].
size_t upd_smem_bytes(int Din, int H) {
  return sizeof(float) * (static_cast<size_t>(kUpdRows) * ((Din + 3) & ~3) + 2 * static_cast<size_t>(kUpdRows) * H +
                          static_cast<size_t>(H) * kUpdTS + kUpdRows * 8 + kUpdRows * 2);
}

struct UpdScratch {
  double *stats, *stat_part, *term_part;
  float *wt, *partial;
  unsigned char *image;  // weight image of the tensor-core paths
  int slices;
};
size_t image_room() {
  const size_t a = ppo_tc_image_bytes(), b = ppo_tc256_image_bytes(kMaxAgents);
  return ((a > b ? a : b) + 255) / 256 * 256;
}
UpdScratch carve(mava_rollout *h, size_t n_params, int slices) {
  unsigned char *p = static_cast<unsigned char *>(h->d_upd);
  UpdScratch s{};
  s.stats = reinterpret_cast<double *>(p); p += 64;
  s.stat_part = reinterpret_cast<double *>(p); p += sizeof(double) * 2 * kStatBlocks;
  s.term_part = reinterpret_cast<double *>(p); p += sizeof(double) * 3 * 8 * slices;
  s.wt = reinterpret_cast<float *>(p); p += sizeof(float) * ((n_params + 3) / 4 * 4);
  s.image = p; p += image_room();
  s.partial = reinterpret_cast<float *>(p);
  s.slices = slices;
  return s;
}

constexpr int kChunkTiles = 4096;  // rows of a chunk of the H = 256 tensor-core path: 524 288 (1.2 GB of staging)

}  // namespace

// A bf16 handle takes the tensor-core kernels for the shapes they serve, unless it asked for the fp32 path.
bool update_takes_tensor_cores(const mava_config_t &cfg, int D) {
  return cfg.precision == MAVA_PRECISION_BF16 && (cfg.flags & MAVA_FLAG_UPDATE_FP32) == 0 && ppo_tc_supported(cfg, D);
}
bool update_takes_tensor_cores_256(const mava_config_t &cfg, int D) {
  return cfg.precision == MAVA_PRECISION_BF16 && (cfg.flags & MAVA_FLAG_UPDATE_FP32) == 0 && ppo_tc256_supported(cfg, D);
}

cudaError_t ensure_update_scratch(mava_rollout *h, size_t n_params, int slices) {
  const size_t bytes = 64 + sizeof(double) * 2 * kStatBlocks + sizeof(double) * 3 * 8 * slices + sizeof(float) * ((n_params + 3) / 4 * 4) +
                       image_room() + sizeof(float) * n_params * slices;
  if (h->d_upd && h->upd_bytes >= bytes) return cudaSuccess;
  cudaFree(h->d_upd);
  h->d_upd = nullptr;
  h->upd_bytes = 0;
  cudaError_t err = cudaMalloc(&h->d_upd, bytes);
  if (err == cudaSuccess) h->upd_bytes = bytes;
  return err;
}

cudaError_t ensure_update_staging(mava_rollout *h, size_t bytes) {
  if (h->d_upd_stage && h->upd_stage_bytes >= bytes) return cudaSuccess;
  cudaFree(h->d_upd_stage);
  h->d_upd_stage = nullptr;
  h->upd_stage_bytes = 0;
  cudaError_t err = cudaMalloc(&h->d_upd_stage, bytes);
  if (err == cudaSuccess) h->upd_stage_bytes = bytes;
  return err;
}

cudaError_t launch_ppo_grad(mava_rollout *h, const float *params_dev, const mava_ppo_hyper_t &hyper, float *grad_dev,
                            float *terms_dev, const int32_t *env_ids_dev, int32_t n_ids) {
  const mava_config_t &cfg = h->cfg;
  const int T = h->last_T, E = cfg.n_envs, N = cfg.n_agents, D = h->D, H = cfg.hidden;
  const ParamLayout L = param_layout(cfg, D, 1);
  const size_t P = L.total;
  int sms = 0;
  cudaError_t err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->device);
  if (err != cudaSuccess) return err;
  const int n_env = env_ids_dev ? n_ids : E;  // environments in the minibatch
  const long long R = static_cast<long long>(T) * n_env * N, S = static_cast<long long>(T) * n_env;
  const long long tiles128 = (R + 127) / 128;
  const bool central = cfg.net_kind == MAVA_NET_CENTRAL_CRITIC;
  const UpdHyper hp{hyper.clip_eps, hyper.ent_coef, hyper.vf_coef};
  cudaStream_t st = h->stream;
  UpdRows rows{};
  rows.x = h->buf.obs; rows.actions = h->buf.actions; rows.logp_old = h->buf.logp; rows.adv = h->buf.adv; rows.n = R;
  rows.env_ids = env_ids_dev; rows.n_ids = n_env; rows.E = E; rows.per_env = N;
  if (!central) { rows.value_old = h->buf.values; rows.ret = h->buf.ret; rows.vstride = 1; }

  if (update_takes_tensor_cores(cfg, D)) {
    // H <= 128: one CTA (= one gradient slice) per SM over tiles of 128 rows
    const int slices = static_cast<int>(tiles128 < sms ? tiles128 : sms);
    err = ensure_update_scratch(h, P, slices);
    if (err != cudaSuccess) return err;
    const UpdScratch sc = carve(h, P, slices);
    stat_partial_kernel<<<kStatBlocks, 256, 0, st>>>(h->buf.adv, R, sc.stat_part, rows);
    stat_final_kernel<<<1, 32, 0, st>>>(sc.stat_part, kStatBlocks, R, sc.stats);
    h->launches += 2;
    err = launch_ppo_net_tc(h, params_dev, L, rows, hp, sc.stats, sc.image, sc.partial, P, sc.term_part, slices);
    if (err != cudaSuccess) return err;
    reduce_partials_kernel<<<128, 256, 0, st>>>(sc.partial, P, slices, grad_dev, sc.term_part, 8 * slices, R, R, hp, terms_dev);
    h->launches += 1;
    return cudaGetLastError();
  }

  // H = 256 on the tensor cores: the actor / shared-torso net and, one input slab per agent, the centralised critic's
  const bool tc256 = update_takes_tensor_cores_256(cfg, D);
  const int min_slices = 1 + (central ? N : 1);  // the weight kernel needs a CTA for d W2 and one per input slab
  const int slices_tc = tc256 ? static_cast<int>(tiles128 < sms ? (tiles128 < min_slices ? min_slices : tiles128) : sms) : 0;
  const long long tiles = (R + kUpdRows - 1) / kUpdRows;
  // fp32 kernel: as many CTAs (= gradient slices) as are resident at once with the larger of the two nets' shared-memory needs
  const int joint = N * D;
  const size_t smem_max = upd_smem_bytes(central ? joint : D, H);
  using KernelT = void (*)(UpdNet, UpdRows, UpdHyper, const double *, float *, size_t, double *, int *);
  const KernelT kern = H == 64 ? ppo_net_kernel<64> : (H == 128 ? ppo_net_kernel<128> : (H == 256 ? ppo_net_kernel<256> : nullptr));
  if (!kern) return cudaErrorNotSupported;
  err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_max));
  if (err != cudaSuccess) return err;
  int per_sm = 1;
  err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, H, smem_max);
  if (err != cudaSuccess) return err;
  if (per_sm < 1) per_sm = 1;
  const int slices_fp32 = static_cast<int>(tiles < static_cast<long long>(sms) * per_sm ? tiles : static_cast<long long>(sms) * per_sm);
  const int slices = slices_fp32 > slices_tc ? slices_fp32 : slices_tc;
  err = ensure_update_scratch(h, P, slices);
  if (err != cudaSuccess) return err;
  const int chunk_tiles = static_cast<int>(tiles128 < kChunkTiles ? tiles128 : kChunkTiles);
  if (tc256) {
    err = ensure_update_staging(h, ppo_tc256_staging_bytes(chunk_tiles, central ? N : 1));
    if (err != cudaSuccess) return err;
  }
  const UpdScratch sc = carve(h, P, slices);
  // transposed copies of the hidden layers' weights, in the parameters' own order (fp32 kernel only)
  auto tr = [&](size_t off, int out, int in) {
    transpose_kernel<<<64, 256, 0, st>>>(params_dev + off, sc.wt + off, out, in);
    h->launches += 1;
  };
  if (!tc256) {
    tr(L.W1, H, D); tr(L.W2, H, H);
    if (central) { tr(L.C1, H, joint); tr(L.C2, H, H); }
  }
  stat_partial_kernel<<<kStatBlocks, 256, 0, st>>>(h->buf.adv, R, sc.stat_part, rows);
  stat_final_kernel<<<1, 32, 0, st>>>(sc.stat_part, kStatBlocks, R, sc.stats);
  h->launches += 2;
  err = cudaMemsetAsync(sc.term_part, 0, sizeof(double) * 3 * 8 * slices, st);
  if (err == cudaSuccess) err = cudaMemsetAsync(sc.partial, 0, sizeof(float) * P * slices, st);
  if (err != cudaSuccess) return err;
  auto run_net = [&](const UpdNet &net, const UpdRows &rows) {
    const size_t smem = upd_smem_bytes(net.Din, net.H);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    kern<<<slices_fp32, net.H, smem, st>>>(net, rows, hp, sc.stats, sc.partial, P, sc.term_part, h->d_status);
    h->launches += 1;
    return cudaGetLastError();
  };
  UpdNet actor{};
  actor.W1 = params_dev + L.W1; actor.b1 = params_dev + L.b1; actor.W2 = params_dev + L.W2; actor.b2 = params_dev + L.b2;
  actor.W1t = sc.wt + L.W1; actor.W2t = sc.wt + L.W2;
  actor.Wa = params_dev + L.Wa; actor.ba = params_dev + L.ba;
  actor.Din = D; actor.H = H;
  actor.oW1 = L.W1; actor.ob1 = L.b1; actor.oW2 = L.W2; actor.ob2 = L.b2; actor.oWa = L.Wa; actor.oba = L.ba;
  if (!central) {
    actor.Wv = params_dev + L.Wv; actor.bv = params_dev + L.bv; actor.oWv = L.Wv; actor.obv = L.bv;
    const Tc256Net net{L.W1, L.b1, L.W2, L.b2, L.Wa, L.ba, L.Wv, L.bv, 1, true, true};
    err = tc256 ? launch_ppo_net_tc256(h, params_dev, net, rows, hp, sc.stats, sc.image, h->d_upd_stage, chunk_tiles, sc.partial, P,
                                       sc.term_part, slices_tc)
                : run_net(actor, rows);
  } else {
    const Tc256Net anet{L.W1, L.b1, L.W2, L.b2, L.Wa, L.ba, 0, 0, 1, true, false};
    err = tc256 ? launch_ppo_net_tc256(h, params_dev, anet, rows, hp, sc.stats, sc.image, h->d_upd_stage, chunk_tiles, sc.partial, P,
                                       sc.term_part, slices_tc)
                : run_net(actor, rows);
    if (err != cudaSuccess) return err;
    UpdNet critic{};
    critic.W1 = params_dev + L.C1; critic.b1 = params_dev + L.c1; critic.W2 = params_dev + L.C2; critic.b2 = params_dev + L.c2;
    critic.W1t = sc.wt + L.C1; critic.W2t = sc.wt + L.C2;
    critic.Wv = params_dev + L.Cv; critic.bv = params_dev + L.cv;
    critic.Din = joint; critic.H = H;
    critic.oW1 = L.C1; critic.ob1 = L.c1; critic.oW2 = L.C2; critic.ob2 = L.c2; critic.oWv = L.Cv; critic.obv = L.cv;
    UpdRows crows{};
    crows.x = h->buf.obs; crows.value_old = h->buf.values; crows.ret = h->buf.ret; crows.vstride = N; crows.n = S;
    crows.env_ids = env_ids_dev; crows.n_ids = n_env; crows.E = E; crows.per_env = 1;
    const Tc256Net cnet{L.C1, L.c1, L.C2, L.c2, 0, 0, L.Cv, L.cv, N, false, true};
    err = tc256 ? launch_ppo_net_tc256(h, params_dev, cnet, crows, hp, sc.stats, sc.image, h->d_upd_stage, chunk_tiles, sc.partial, P,
                                       sc.term_part, slices_tc)
                : run_net(critic, crows);
  }
  if (err != cudaSuccess) return err;
  reduce_partials_kernel<<<128, 256, 0, st>>>(sc.partial, P, slices, grad_dev, sc.term_part, 8 * slices, R, central ? S : R, hp,
                                              terms_dev);
  h->launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_adam_step(mava_rollout *h, float *params_dev, const float *grad_dev, float *m_dev, float *v_dev, int32_t step,
                             const mava_ppo_hyper_t &hp) {
  const size_t P = param_layout(h->cfg, h->D, 1).total;
  cudaError_t err = ensure_update_scratch(h, P, 1);
  if (err != cudaSuccess) return err;
  const UpdScratch sc = carve(h, P, 1);
  stat_partial_kernel<<<kStatBlocks, 256, 0, h->stream>>>(grad_dev, static_cast<long long>(P), sc.stat_part, UpdRows{});
  stat_final_kernel<<<1, 32, 0, h->stream>>>(sc.stat_part, kStatBlocks, static_cast<long long>(P), sc.stats);
  const float corr1 = static_cast<float>(1.0 - pow(static_cast<double>(hp.beta1), step));
  const float corr2 = static_cast<float>(1.0 - pow(static_cast<double>(hp.beta2), step));
  adam_kernel<<<128, 256, 0, h->stream>>>(params_dev, grad_dev, m_dev, v_dev, P, sc.stats, hp.max_grad_norm, hp.lr, hp.beta1, hp.beta2,
                                          hp.adam_eps, corr1, corr2);
  h->launches += 3;
  return cudaGetLastError();
}

}  // namespace mava
