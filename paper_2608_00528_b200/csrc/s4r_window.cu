// Windowed relevance estimation (Eq. 7, 9, 10): instead of the current query alone, the W_q most recent
// projected queries score the cache, each under its own causal limit, and their probabilities are averaged.
//
// The query-coefficient window is caller-owned state [B][W_q][G][r_k] fp32, oldest row first.  A step shifts it
// by one row and appends the current query's coefficients; the same kernel (k_window_prepare) also writes the
// window as the tensor-core operand the scoring kernels copy into shared memory: per sequence and per set of
// query groups scored together, two bf16 terms (hi, mid) of [r_k / 64][128 rows][64 columns], K-major with the
// 128-byte swizzle, row (g - g0) W_q + i for window row i of group g, unused rows zero.  The windowed scoring
// kernels then score every row, average the probabilities per query group and hand the logarithm of that
// average to the relevance kernel, which pools, aggregates and bins it exactly as it does for a single query
// (its "softmax" of ln(a) with normaliser 1 returns a).
#include "s4r_internal.h"
#include "s4r_sm100.cuh"

namespace s4r {

namespace {

constexpr int kWinThreads = 128;
constexpr int kPieceBytes = 128 * 128;

struct WinPrepParams {
  float *window;     // [B][W_q][G][r]
  const float *cq;   // [B][G][r]: the current query's coefficients
  uint8_t *wimg;     // [sets][B][2][r / 64][128][128 B]
  int B, Wq, G, r, gpl, sets;
};

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(a)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(b)) << 16);
}

// A thread owns two adjacent columns (g, k), (g, k + 1) of the window, so the in-place shift has no hazard.
__global__ void __launch_bounds__(kWinThreads) k_window_prepare(WinPrepParams p) {
  grid_dependency_sync();
  const int b = blockIdx.x;
  const int n = p.G * p.r;
  const size_t term_bytes = (size_t)(p.r >> 6) * kPieceBytes, image_bytes = 2 * term_bytes;
  float *w = p.window + (size_t)b * p.Wq * n;
  const int x = 2 * (blockIdx.y * kWinThreads + threadIdx.x);
  if (x < n) {
    const int g = x / p.r, k = x - g * p.r;
    const int set = g / p.gpl, gl = g - set * p.gpl;
    uint8_t *img = p.wimg + ((size_t)set * p.B + b) * image_bytes + (size_t)(k >> 6) * kPieceBytes;
    const int row0 = gl * p.Wq;
    const float2 newest = *reinterpret_cast<const float2 *>(p.cq + (size_t)b * n + x);
    // sixteen rows per trip to memory: rows i0 + 1 .. i0 + 16 are read before rows i0 .. i0 + 15 are written
    for (int i0 = 0; i0 < p.Wq; i0 += 16) {
      float2 t[16];
#pragma unroll
      for (int q = 0; q < 16; ++q)
        if (i0 + q + 1 < p.Wq) t[q] = *reinterpret_cast<const float2 *>(w + (size_t)(i0 + q + 1) * n + x);
#pragma unroll
      for (int q = 0; q < 16; ++q) {
        const int i = i0 + q;
        if (i < p.Wq) {
          const float2 v = i + 1 < p.Wq ? t[q] : newest;
          *reinterpret_cast<float2 *>(w + (size_t)i * n + x) = v;
          const __nv_bfloat16 h0 = __float2bfloat16_rn(v.x), h1 = __float2bfloat16_rn(v.y);
          const uint32_t off = sm100::sw128_offset(row0 + i, k & 63);
          *reinterpret_cast<uint32_t *>(img + off) =
              (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
          *reinterpret_cast<uint32_t *>(img + term_bytes + off) =
              pack_bf16(v.x - __bfloat162float(h0), v.y - __bfloat162float(h1));
        }
      }
    }
  }
  // rows of the images that carry no window row: 16-byte pieces, spread over the sequence's thread blocks
  const int kb2 = 2 * (p.r >> 6);
  for (int set = 0; set < p.sets; ++set) {
    const int ng = min(p.gpl, p.G - set * p.gpl);
    const int R = ng * p.Wq, n_zero = (128 - R) * 8 * kb2;
    uint8_t *img = p.wimg + ((size_t)set * p.B + b) * image_bytes;
    for (int idx = blockIdx.y * kWinThreads + threadIdx.x; idx < n_zero; idx += gridDim.y * kWinThreads) {
      const int piece = idx & 7, rest = idx >> 3;
      const int row = R + rest % (128 - R), blk = rest / (128 - R);
      *reinterpret_cast<uint4 *>(img + (size_t)blk * kPieceBytes + (size_t)(row >> 3) * 1024 + (row & 7) * 128 + piece * 16) =
          make_uint4(0, 0, 0, 0);
    }
  }
}

}  // namespace

cudaError_t launch_window_prepare(float *window, const float *cq, uint8_t *wimg, const Layer &ly, int Wq, int gpl,
                                  int sets, cudaStream_t st) {
  WinPrepParams p;
  p.window = window; p.cq = cq; p.wimg = wimg; p.B = ly.B; p.Wq = Wq; p.G = ly.G; p.r = ly.rk; p.gpl = gpl; p.sets = sets;
  const int n = ly.G * ly.rk;
  dim3 grid(ly.B, (n / 2 + kWinThreads - 1) / kWinThreads);
  cudaError_t e = launch_chained(k_window_prepare, grid, dim3(kWinThreads), 0, st, 1, p);
  if (e != cudaSuccess) return e;
  ++launch_counter();
  return cudaGetLastError();
}

}  // namespace s4r
