// Windowed relevance estimation (Eq. 7, 9, 10): instead of the current query alone, the W_q most recent
// projected queries score the cache, each under its own causal limit, and their probabilities are averaged.
//
// The query-coefficient window is caller-owned state [B][W_q][G][r_k] fp32, oldest row first.  A step shifts it
// by one row and appends the current query's coefficients (k_window_shift), scores every row with the scan
// kernel in blocks of up to eight rows, averages the probabilities per query group (k_window_mean) and hands
// the logarithm of that average to the relevance kernel, which then pools, aggregates and bins it exactly as it
// does for a single query (its "softmax" of ln(a) with normaliser 1 returns a).
#include "s4r_internal.h"

namespace s4r {

namespace {

constexpr int kWinThreads = 256;

// window[b][i] <- window[b][i + 1], last row <- the current query's coefficients.  A thread owns a column, so
// the in-place shift has no hazard.
__global__ void __launch_bounds__(kWinThreads) k_window_shift(float *window, const float *cq, int Wq, int n) {
  grid_dependency_sync();
  const int b = blockIdx.x;
  float *w = window + (size_t)b * Wq * n;
  for (int x = threadIdx.x; x < n; x += kWinThreads) {
    for (int i = 0; i + 1 < Wq; ++i) w[(size_t)i * n + x] = w[(size_t)(i + 1) * n + x];
    w[(size_t)(Wq - 1) * n + x] = cq[(size_t)b * n + x];
  }
}

struct WinMeanParams {
  const float *Z;        // [B][rows_alloc][z_stride]: row rho = i * G + g of the window
  const float2 *part;    // [blocks][B][parts_cap][kMaxGroup]
  const int32_t *coef_len;
  float *zmean;          // [B][G][z_stride]: ln of the window-averaged probability
  float2 *unit;          // [B][kMaxGroup]: (0, 1), the relevance kernel's normalisers for zmean
  int G, Wq, n_parts, parts_cap, rows_alloc, B;
  int64_t max_len, z_stride;
};

__global__ void __launch_bounds__(kWinThreads) k_window_mean(WinMeanParams p) {
  grid_dependency_sync();
  __shared__ float s_c[kMaxScoreRows];  // p = exp2(z * log2e + c), c = -M log2e - log2(S W_q)
  const int b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int L = p.coef_len[b];
  L = L < 0 ? 0 : ((int64_t)L > p.max_len ? (int)p.max_len : L);
  const int R = p.G * p.Wq;
  if (blockIdx.x == 0 && tid < kMaxGroup) p.unit[(size_t)b * kMaxGroup + tid] = make_float2(0.f, 1.f);
  // ---- normalisers of every window row (Eq. 9) from the scan's partials (empty partials are (-inf, 0))
  for (int rho = warp; rho < R; rho += kWinThreads / 32) {
    // block stride as allocated (B * parts_cap), sequence stride as the scan kernel writes it (n_parts)
    const float2 *pp = p.part + ((size_t)(rho >> 3) * p.B * p.parts_cap + (size_t)b * p.n_parts) * kMaxGroup + (rho & 7);
    float m = -INFINITY, s = 0.f;
    for (int c = lane; c < p.n_parts; c += 32) {
      const float2 v = __ldcg(pp + (size_t)c * kMaxGroup);
      if (v.y > 0.f) ms_merge(m, s, v.x, v.y);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
      ms_merge(m, s, m2, s2);
    }
    if (lane == 0) s_c[rho] = s > 0.f ? -m * 1.4426950408889634f - log2f(s * (float)p.Wq) : -INFINITY;
  }
  __syncthreads();
  const int pos = (blockIdx.x * kWinThreads + tid) * 4;
  if (pos >= L) return;
  const float *zb = p.Z + (size_t)b * p.rows_alloc * p.z_stride;
  for (int g = 0; g < p.G; ++g) {
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int i = 0; i < p.Wq; ++i) {
      const int rho = i * p.G + g;
      const int last = L - p.Wq + i;  // window row i belongs to the token at index `last` and sees l <= last
      if (last < pos) continue;
      const float c = s_c[rho];
      const float4 z = __ldcg(reinterpret_cast<const float4 *>(zb + (size_t)rho * p.z_stride + pos));
      const float zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (pos + j <= last) acc[j] += exp2f(fmaf(zz[j], 1.4426950408889634f, c));
    }
    float *dst = p.zmean + ((size_t)b * p.G + g) * p.z_stride + pos;
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (pos + j < L) dst[j] = logf(acc[j]);  // ln 0 = -inf: the position then carries no probability
  }
}

}  // namespace

cudaError_t launch_window_shift(float *window, const float *cq, int B, int Wq, int n, cudaStream_t st) {
  cudaError_t e = launch_chained(k_window_shift, dim3(B), dim3(kWinThreads), 0, st, 1, window, cq, Wq, n);
  if (e != cudaSuccess) return e;
  ++launch_counter();
  return cudaGetLastError();
}

cudaError_t launch_window_mean(const StepArgs &a, const float *Z, const float2 *part, float *zmean, float2 *unit,
                               int Wq, int rows_alloc) {
  if (a.plan.max_len <= 0) return cudaSuccess;
  WinMeanParams p;
  p.Z = Z; p.part = part; p.coef_len = a.coef_len; p.zmean = zmean; p.unit = unit;
  p.G = a.ly.G; p.Wq = Wq; p.n_parts = a.plan.n_parts; p.parts_cap = a.plan.parts_cap; p.rows_alloc = rows_alloc;
  p.B = a.ly.B; p.max_len = a.plan.max_len; p.z_stride = a.plan.z_stride;
  dim3 grid((unsigned)((a.plan.max_len + 4 * kWinThreads - 1) / (4 * kWinThreads)), a.ly.B);
  cudaError_t e = launch_chained(k_window_mean, grid, dim3(kWinThreads), 0, a.stream, 1, p);
  if (e != cudaSuccess) return e;
  ++launch_counter();
  return cudaGetLastError();
}

}  // namespace s4r
