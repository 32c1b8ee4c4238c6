// Latent scoring (Eq. 8) for bf16 coefficient caches on sm_100a: the HBM-bound scan of the decode step.
//
// One CTA streams a contiguous range of 128-row tiles of one sequence's key-coefficient cache through a
// multi-stage TMA pipeline (128-byte swizzled tiles, one mbarrier pair per stage).  Each tile is multiplied
// on the tensor cores (tcgen05.mma, M = 128 tokens, N = 32, K = r) with the projected queries, which are
// held in shared memory as three bf16 terms per value (hi + mid + lo = the fp32 value to 24 bits), so the
// products are exact and the logits keep fp32 accuracy.  Accumulators live in tensor memory (two buffers of
// 32 columns); four epilogue warps read them back, scale by 1/sqrt(r), store Z[b][g][row] and keep the
// running (max, sum exp) of Eq. 9 for the CTA's rows.  Warp 0 = TMA producer, warp 1 = MMA issuer,
// warps 2-5 = epilogue.  grid (CTAs per sequence, B).
#include "s4r_internal.h"
#include "s4r_sm100.cuh"

namespace s4r {

using namespace sm100;

namespace {

constexpr int kTileRows = 128;
constexpr int kScanThreads = 192;
constexpr int kAccCols = 32;  // accumulator columns per buffer: [hi | mid | lo | 0] x 8 group members

struct ScanFastParams {
  const float *cq_part;
  const int32_t *coef_len;
  float *Z;
  float2 *part;
  int r, G, cps, stages;
  int64_t cap, max_len, z_stride;
  float inv_sqrt_r;
  int32_t *dev_status;
};

__device__ __forceinline__ void online_update(float &m, float &s, float z) {
  if (z <= m) {
    s += __expf(z - m);
  } else {
    s = s * __expf(m - z) + 1.f;
    m = z;
  }
}

__global__ void __launch_bounds__(kScanThreads, 1) k_scan_sm100(const __grid_constant__ CUtensorMap tmap,
                                                                ScanFastParams p) {
  grid_dependency_sync();
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int kblocks = p.r >> 6;                    // 64-column blocks per row
  const uint32_t tile_bytes = (uint32_t)kblocks * kTileRows * 128u;
  uint8_t *a_tiles = smem;                                         // [stages][kblocks][128 rows][128 B]
  uint8_t *b_op = a_tiles + (size_t)p.stages * tile_bytes;         // [kblocks][32 rows][128 B]
  uint64_t *bars = reinterpret_cast<uint64_t *>(b_op + (size_t)kblocks * kAccCols * 128);
  uint64_t *full = bars, *empty = bars + p.stages, *acc_full = bars + 2 * p.stages, *acc_empty = acc_full + 2;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  float2 *red = reinterpret_cast<float2 *>(tmem_slot + 4);       // [4 warps][kMaxGroup]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = blockIdx.y, j = blockIdx.x;
  int L = p.coef_len[b];
  if (L < 0 || (int64_t)L > p.max_len) {
    if (p.dev_status && tid == 0) atomicOr(p.dev_status, S4R_DEV_BOUNDS);
    L = L < 0 ? 0 : (int)p.max_len;
  }
  const int tiles_total = (L + kTileRows - 1) / kTileRows;
  const int tpc = (tiles_total + p.cps - 1) / p.cps;
  const int t_begin = min(tiles_total, j * tpc), t_end = min(tiles_total, t_begin + tpc);
  const int n_tiles = t_end - t_begin;
  if (n_tiles <= 0) {  // uniform over the CTA: nothing to scan
    if (tid < p.G) p.part[((size_t)b * p.cps + j) * kMaxGroup + tid] = make_float2(-INFINITY, 0.f);
    return;
  }

  if (tid == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&acc_full[a], 1);
      mbar_init(&acc_empty[a], 4);  // one arrival per epilogue warp
    }
    *abort_flag = 0;
    mbar_fence_init();
    prefetch_tmap(&tmap);
  }
  if (warp == 1) tmem_alloc(tmem_slot, 2 * kAccCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp != 0) {
    // While the producer (warp 0) already streams tiles, the other warps build the B operand: row n = t*8 + g
    // holds term t (0 hi, 1 mid, 2 lo, 3 zero) of c^Q[g], K-major, 128-byte swizzle.  Loads go out in batches
    // of 8 so that their latencies overlap.
    constexpr int kWorkers = kScanThreads - 32;
    const int n_el = kMaxGroup * p.r;
    for (int i0 = tid - 32; i0 < n_el; i0 += 8 * kWorkers) {
      float cval[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int i = i0 + u * kWorkers;
        const int g = i / p.r, k = i - g * p.r;
        cval[u] = (i < n_el && g < p.G) ? __ldcg(p.cq_part + ((size_t)b * p.G + g) * p.r + k) : 0.f;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int i = i0 + u * kWorkers;
        if (i < n_el) {
          const int g = i / p.r, k = i - g * p.r;
          const float c = cval[u];
          const __nv_bfloat16 hi = __float2bfloat16_rn(c);
          const float r1 = c - __bfloat162float(hi);
          const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
          const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
          uint8_t *blk = b_op + (size_t)(k >> 6) * (kAccCols * 128);
          const int kc = k & 63;
          *reinterpret_cast<__nv_bfloat16 *>(blk + sw128_offset(g, kc)) = hi;
          *reinterpret_cast<__nv_bfloat16 *>(blk + sw128_offset(8 + g, kc)) = mid;
          *reinterpret_cast<__nv_bfloat16 *>(blk + sw128_offset(16 + g, kc)) = lo;
          *reinterpret_cast<__nv_bfloat16 *>(blk + sw128_offset(24 + g, kc)) = __float2bfloat16_rn(0.f);
        }
      }
    }
    fence_proxy_async_smem();
    asm volatile("bar.sync 1, %0;" ::"n"(kScanThreads - 32) : "memory");  // B operand complete (producer not involved)
  }

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      const uint64_t pol = policy_evict_first();
      int issued = 0;
      for (int it = 0; it < n_tiles; ++it) {
        const int s = it % p.stages;
        const uint32_t ph = (uint32_t)(it / p.stages) & 1u;
        if (!mbar_wait(&empty[s], ph ^ 1u, abort_flag)) break;
        mbar_expect_tx(&full[s], tile_bytes);
        const int y = (int)((int64_t)b * p.cap) + (t_begin + it) * kTileRows;
        for (int kb = 0; kb < kblocks; ++kb)
          tma_load_2d_hint(a_tiles + (size_t)s * tile_bytes + (size_t)kb * (kTileRows * 128), &tmap, kb * 64, y,
                           &full[s], pol);
        issued = it + 1;
      }
      if (*abort_flag) {  // drain: do not leave while bulk copies may still land in this CTA's shared memory
        for (int it = max(0, issued - p.stages); it < issued; ++it) {
          const unsigned long long t0 = global_ns();
          while (!mbar_try_wait(&full[it % p.stages], (uint32_t)(it / p.stages) & 1u))
            if (global_ns() - t0 > kWaitLimitNs) break;
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(kTileRows, kAccCols);
      const uint64_t b_desc0 = umma_desc_sw128(smem_u32(b_op));
      for (int it = 0; it < n_tiles; ++it) {
        const int s = it % p.stages, a = it & 1;
        const uint32_t ph = (uint32_t)(it / p.stages) & 1u, aph = (uint32_t)(it >> 1) & 1u;
        if (!mbar_wait(&acc_empty[a], aph ^ 1u, abort_flag)) break;
        if (!mbar_wait(&full[s], ph, abort_flag)) break;
        tc_fence_after();
        const uint64_t a_desc0 = umma_desc_sw128(smem_u32(a_tiles + (size_t)s * tile_bytes));
        const uint32_t d_tmem = tmem_base + (uint32_t)a * kAccCols;
        for (int kb = 0; kb < kblocks; ++kb) {
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4) {
            const uint64_t a_desc = a_desc0 + (uint64_t)((kb * (kTileRows * 128) + k4 * 32) >> 4);
            const uint64_t b_desc = b_desc0 + (uint64_t)((kb * (kAccCols * 128) + k4 * 32) >> 4);
            umma_bf16(d_tmem, a_desc, b_desc, idesc, (kb | k4) != 0);
          }
        }
        umma_commit(&empty[s]);      // the stage is free once these MMAs have read it
        umma_commit(&acc_full[a]);   // and the accumulator is ready
      }
    }
  } else {
    // ---------------- epilogue: 4 warps, one TMEM lane quadrant each ----------------
    const int quad = warp & 3;
    const int row_in_tile = quad * 32 + lane;
    float m[kMaxGroup], sm[kMaxGroup];
#pragma unroll
    for (int g = 0; g < kMaxGroup; ++g) {
      m[g] = -INFINITY;
      sm[g] = 0.f;
    }
    float *zb = p.Z + (size_t)b * p.G * p.z_stride;
    for (int it = 0; it < n_tiles; ++it) {
      const int a = it & 1;
      const uint32_t aph = (uint32_t)(it >> 1) & 1u;
      if (!mbar_wait(&acc_full[a], aph, abort_flag)) break;
      tc_fence_after();
      uint32_t v[32];
      tmem_ld32(tmem_base + (uint32_t)a * kAccCols + ((uint32_t)(quad * 32) << 16), v);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[a]);
      const int row = (t_begin + it) * kTileRows + row_in_tile;
      if (row < L) {
#pragma unroll
        for (int g = 0; g < kMaxGroup; ++g) {
          if (g < p.G) {
            const float z = ((__uint_as_float(v[16 + g]) + __uint_as_float(v[8 + g])) + __uint_as_float(v[g])) *
                            p.inv_sqrt_r;
            zb[(size_t)g * p.z_stride + row] = z;
            online_update(m[g], sm[g], z);
          }
        }
      }
    }
#pragma unroll
    for (int g = 0; g < kMaxGroup; ++g) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m[g], o);
        const float s2 = __shfl_xor_sync(0xffffffffu, sm[g], o);
        ms_merge(m[g], sm[g], m2, s2);
      }
      if (lane == 0) red[quad * kMaxGroup + g] = make_float2(m[g], sm[g]);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (tid < p.G) {
    float mm = -INFINITY, ss = 0.f;
    for (int w = 0; w < 4; ++w) {
      const float2 v = red[w * kMaxGroup + tid];
      ms_merge(mm, ss, v.x, v.y);
    }
    p.part[((size_t)b * p.cps + j) * kMaxGroup + tid] = make_float2(mm, ss);
  }
  if (tid == 0 && *abort_flag && p.dev_status) atomicOr(p.dev_status, S4R_DEV_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 2 * kAccCols);
  }
}

}  // namespace

// ---- host: tensor map encode through the driver entry point (no link-time dependency on libcuda) ----------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool make_tmap_bf16_2d(CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !sym)
      return false;
    fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  const cuuint64_t gdim[2] = {cols, rows};
  const cuuint64_t gstride[1] = {cols * 2};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool scan_fast_supported(const Layer &ly) {
  return ly.dtype == S4R_BF16 && ly.rk % 64 == 0 && ly.rk >= 64 && ly.rk <= 512 && ly.cap > 0 &&
         (int64_t)ly.B * ly.cap < 0x7fffffffLL - 256;
}

int scan_fast_parts(const Layer &ly) {
  static int sms = 0;
  if (!sms) {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      return 0;
    sms = n;
  }
  int cps = sms / ly.B;
  if (cps < 1) cps = 1;
  if (cps > kMaxParts) cps = kMaxParts;
  return cps;
}

cudaError_t launch_scan_sm100(const StepArgs &a) {
  const Layer &ly = a.ly;
  CUtensorMap tmap;
  if (!make_tmap_bf16_2d(&tmap, a.coef_k, (uint64_t)ly.B * (uint64_t)ly.cap, (uint64_t)ly.rk, kTileRows))
    return cudaErrorInvalidValue;
  ScanFastParams p;
  p.cq_part = (const float *)(a.ws + a.plan.off_cq);
  p.coef_len = a.coef_len;
  p.Z = (float *)(a.ws + a.plan.off_z);
  p.part = (float2 *)(a.ws + a.plan.off_part);
  p.r = ly.rk;
  p.G = ly.G;
  p.cps = a.plan.n_parts;
  p.cap = ly.cap;
  p.max_len = a.plan.max_len;
  p.z_stride = a.plan.z_stride;
  p.inv_sqrt_r = (float)(1.0 / sqrt((double)ly.rk));
  p.dev_status = a.dev_status;
  const size_t tile_bytes = (size_t)(ly.rk / 64) * kTileRows * 128;
  const size_t fixed = (size_t)(ly.rk / 64) * kAccCols * 128 + 1024 /*alignment*/ + 1024 /*barriers, flags, red*/;
  int stages = (int)((226 * 1024 - fixed) / tile_bytes);
  if (stages > 8) stages = 8;
  if (stages < 2) return cudaErrorInvalidValue;
  p.stages = stages;
  const size_t smem = fixed + (size_t)stages * tile_bytes;
  static size_t smem_set = 0;
  if (smem > smem_set) {
    cudaError_t e = cudaFuncSetAttribute(k_scan_sm100, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    smem_set = smem;
  }
  dim3 grid(p.cps, ly.B);
  cudaError_t le = launch_chained(k_scan_sm100, grid, dim3(kScanThreads), smem, a.stream, 1, tmap, p);
  if (le != cudaSuccess) return le;
  ++launch_counter();
  return cudaGetLastError();
}

}  // namespace s4r
