// Dense layer of the fp32 SIMT kernels over a tile of rows held in shared memory.
#pragma once
#include "common.cuh"

namespace mava {

constexpr int kSimtThreads = 256;
constexpr int kSimtRows = 32;  // agent rows per tile (upper bound; a tile holds floor(32/N) envs)

// y[row][o] = act(sum_k x[row][k] * Wt[k][o] + b[o]) for `ROWS` rows held in shared memory.
// Thread (rg, cg) owns four consecutive outputs of RPT rows; k runs in ascending order.
template <int K, int HOUT, int ROWS, bool RELU>
__device__ __forceinline__ void dense_tile(const float *xs, int x_stride, const float *__restrict__ Wt,
                                           const float *__restrict__ b, float *ys, int y_stride, int tid) {
  constexpr int CG = HOUT / 4;
  constexpr int RG = kSimtThreads / CG;
  constexpr int RPT = (ROWS + RG - 1) / RG;
  static_assert(kSimtThreads % CG == 0, "thread layout");
  const int cg = tid % CG, rg = tid / CG;
  float acc[RPT][4];
#pragma unroll
  for (int i = 0; i < RPT; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.0f;
  for (int k = 0; k < K; ++k) {
    const float4 w = __ldg(reinterpret_cast<const float4 *>(Wt + static_cast<size_t>(k) * HOUT) + cg);
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
      const int row = rg + i * RG;
      const float x = row < ROWS ? xs[row * x_stride + k] : 0.0f;
      acc[i][0] = fmaf(x, w.x, acc[i][0]);
      acc[i][1] = fmaf(x, w.y, acc[i][1]);
      acc[i][2] = fmaf(x, w.z, acc[i][2]);
      acc[i][3] = fmaf(x, w.w, acc[i][3]);
    }
  }
  const float4 bias = __ldg(reinterpret_cast<const float4 *>(b) + cg);
#pragma unroll
  for (int i = 0; i < RPT; ++i) {
    const int row = rg + i * RG;
    if (row >= ROWS) continue;
    float v0 = acc[i][0] + bias.x, v1 = acc[i][1] + bias.y, v2 = acc[i][2] + bias.z, v3 = acc[i][3] + bias.w;
    if (RELU) { v0 = fmaxf(v0, 0.0f); v1 = fmaxf(v1, 0.0f); v2 = fmaxf(v2, 0.0f); v3 = fmaxf(v3, 0.0f); }
    float *y = ys + row * y_stride + cg * 4;
    y[0] = v0; y[1] = v1; y[2] = v2; y[3] = v3;
  }
}

}  // namespace mava
