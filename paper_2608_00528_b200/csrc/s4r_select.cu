// Relevance + selection (Eq. 9-15).  One thread-block cluster per sequence; each CTA owns a contiguous
// slice of the cache and keeps its scores in shared memory.
//
//   1. softmax normalisers of Eq. 9 from the scan kernel's (max, sum exp) partials;
//   2. score[l] = F_G over g of pool_kappa(softmax_g)[l]  (Eq. 11-12), 4096 positions per pass;
//   3. scores are probabilities (>= 0), so their fp32 bit patterns order like the values: the k-th largest
//      candidate is found exactly by a 3-pass radix select (11 + 11 + 10 bits) whose histograms are summed
//      across the cluster through distributed shared memory;
//   4. winners are written in ascending index order (equal scores: lower index first) by warp-level
//      ballots; the local window of Eq. 13 is appended behind them.
#include <cooperative_groups.h>

#include "s4r_internal.h"

namespace cg = cooperative_groups;

namespace s4r {

namespace {

constexpr int kHalo = 16;
constexpr int kSelTile = 4 * kSelThreads;   // positions per scoring pass
constexpr int kSliceCap = 16384;            // scores of a slice kept in shared memory up to this many

struct SelParams {
  const float *Z;
  const float2 *part;
  const int32_t *coef_len;
  float *score;
  int32_t *sel_idx, *sel_count;
  int G, n_parts, window, top_k, kappa, pool_mode, group_mode;
  int64_t max_len, z_stride;
  int32_t *dev_status;
};

// exclusive prefix sum over the block; total in *total
__device__ inline unsigned block_excl_scan(unsigned v, unsigned *s_warp, unsigned *total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    unsigned t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    unsigned w = s_warp[lane];
    unsigned winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      unsigned t = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += t;
    }
    s_warp[lane] = winc - w;
    if (lane == 31) s_warp[32] = winc;
  }
  __syncthreads();
  unsigned res = s_warp[warp] + inc - v;
  *total = s_warp[32];
  __syncthreads();
  return res;
}

// Sum the per-CTA histograms of the cluster and locate the bin that holds the k_rem-th largest element
// (bins are scanned from the top).  Every CTA pushes its non-empty bins into rank 0's `s_tot` with remote
// atomics (no remote reads, so nobody waits on distributed-shared-memory latency); rank 0 scans the totals,
// writes (bin, elements above it) into every CTA's `s_bc` and clears `s_tot` for the next round.
// Returns the bin; *above = number of elements in higher bins.
__device__ inline unsigned find_bin(cg::cluster_group &cluster, unsigned *s_hist, unsigned *s_tot, unsigned *s_warp,
                                    unsigned *s_bc, int nbins, unsigned k_rem, unsigned *above) {
  const int CL = cluster.num_blocks();
  const int t = threadIdx.x;
  __syncthreads();  // this CTA's histogram is complete
  {
    unsigned *tot0 = cluster.map_shared_rank(s_tot, 0);
    for (int i = t; i < nbins; i += kSelThreads) {
      const unsigned c = s_hist[i];
      if (c) atomicAdd(&tot0[i], c);
    }
  }
  cluster.sync();  // all pushes have landed
  if (cluster.block_rank() == 0) {
    const int b0 = nbins - 1 - 2 * t, b1 = nbins - 2 - 2 * t;
    const unsigned c0 = b0 >= 0 ? s_tot[b0] : 0u, c1 = b1 >= 0 ? s_tot[b1] : 0u;
    unsigned total;
    const unsigned excl = block_excl_scan(c0 + c1, s_warp, &total);
    unsigned found = 0xffffffffu, abv = 0;
    if (b0 >= 0 && excl < k_rem && k_rem <= excl + c0) {
      found = (unsigned)b0;
      abv = excl;
    } else if (b1 >= 0 && excl + c0 < k_rem && k_rem <= excl + c0 + c1) {
      found = (unsigned)b1;
      abv = excl + c0;
    }
    if (found != 0xffffffffu) {
      for (int rk = 0; rk < CL; ++rk) {
        unsigned *bc = cluster.map_shared_rank(s_bc, rk);
        bc[0] = found;
        bc[1] = abv;
      }
    }
    if (b0 >= 0) s_tot[b0] = 0;
    if (b1 >= 0) s_tot[b1] = 0;
  }
  cluster.sync();  // result delivered, totals cleared
  *above = s_bc[1];
  return s_bc[0];
}

__global__ void __launch_bounds__(kSelThreads, 1) k_select(SelParams p) {
  cg::cluster_group cluster = cg::this_cluster();
  const int CL = cluster.num_blocks();
  const int rank = cluster.block_rank();
  const int b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  extern __shared__ __align__(16) float dsm[];
  float *s_score = dsm;                 // [kSliceCap]
  float *s_p = dsm + kSliceCap;         // [G][kSelTile + 2 * kHalo]
  constexpr int kRow = kSelTile + 2 * kHalo;
  __shared__ unsigned s_hist[2048];
  __shared__ unsigned s_tot[2048];      // cluster-wide histogram, used in rank 0 only
  __shared__ unsigned s_cnts[kMaxCluster][2];  // (greater, equal) counts of the lower-ranked CTAs
  __shared__ float s_M[kMaxGroup], s_iS[kMaxGroup];
  __shared__ unsigned s_warp[33];
  __shared__ unsigned s_bc[2];
  __shared__ unsigned s_wcnt[32][2];

  int L = p.coef_len[b];
  if (L < 0 || (int64_t)L > p.max_len) {
    if (p.dev_status && tid == 0) atomicOr(p.dev_status, S4R_DEV_BOUNDS);
    L = L < 0 ? 0 : (int)p.max_len;
  }
  const int W_eff = min(p.window, L);
  const int n_cand = L - W_eff;
  const int k_eff = min(p.top_k, n_cand);
  int32_t *out_idx = p.sel_idx + (size_t)b * (p.window + p.top_k);

  if (rank == 0) {  // local window (Eq. 13), padding and count
    for (int j = tid; j < W_eff; j += kSelThreads) out_idx[k_eff + j] = n_cand + j;
    for (int j = k_eff + W_eff + tid; j < p.window + p.top_k; j += kSelThreads) out_idx[j] = -1;
    if (tid == 0) p.sel_count[b] = k_eff + W_eff;
  }
  if (k_eff == 0) return;  // uniform over the cluster: nothing to rank

  // ---- softmax normalisers of Eq. 9 from the scan's partials (empty partials are (-inf, 0))
  if (warp < p.G) {
    const float2 *pp = p.part + (size_t)b * p.n_parts * kMaxGroup + warp;
    float m = -INFINITY;
    for (int c = lane; c < p.n_parts; c += 32) m = fmaxf(m, pp[(size_t)c * kMaxGroup].x);
    m = warp_max(m);
    float s = 0.f;
    for (int c = lane; c < p.n_parts; c += 32) {
      float2 v = pp[(size_t)c * kMaxGroup];
      if (v.y > 0.f) s += v.y * expf(v.x - m);
    }
    s = warp_sum(s);
    if (lane == 0) {
      s_M[warp] = m;
      s_iS[warp] = 1.f / s;
    }
  }
  for (int i = tid; i < 2048; i += kSelThreads) {
    s_hist[i] = 0;
    s_tot[i] = 0;
  }
  cluster.sync();  // rank 0's totals are clear before anybody pushes into them

  // ---- scores of this CTA's slice (Eq. 9-12) + first histogram
  int per = (L + CL - 1) / CL;
  per = (per + 3) & ~3;
  const int begin = min(L, rank * per), end = min(L, begin + per);
  const int half = p.kappa >> 1;
  const float *zb = p.Z + (size_t)b * p.G * p.z_stride;
  float *score = (per <= kSliceCap) ? s_score : p.score + (size_t)b * p.z_stride + begin;  // indexed by l - begin
  const float inv_kappa = 1.f / (float)p.kappa, inv_G = 1.f / (float)p.G;
  for (int l0 = begin; l0 < end; l0 += kSelTile) {
    {
      // all loads of the pass are issued before anything is stored, so they overlap
      const int l = l0 + 4 * tid;
      const bool vec = l + 3 < L;
      const int side = (tid >> 4) & 1, hj = tid & 15;
      const int lh = side ? l0 + kSelTile + hj : l0 - kHalo + hj;
      const bool halo_ok = tid < 2 * kHalo && lh >= 0 && lh < L;
      float4 z[kMaxGroup];
      float zh[kMaxGroup];
#pragma unroll
      for (int g = 0; g < kMaxGroup; ++g) {
        z[g] = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        zh[g] = -INFINITY;
        if (g < p.G) {
          const float *zr = zb + (size_t)g * p.z_stride;
          if (vec) {
            z[g] = __ldcg(reinterpret_cast<const float4 *>(zr + l));
          } else {
            if (l < L) z[g].x = __ldcg(zr + l);
            if (l + 1 < L) z[g].y = __ldcg(zr + l + 1);
            if (l + 2 < L) z[g].z = __ldcg(zr + l + 2);
          }
          if (halo_ok) zh[g] = __ldcg(zr + lh);
        }
      }
#pragma unroll
      for (int g = 0; g < kMaxGroup; ++g) {
        if (g < p.G) {
          const float M = s_M[g], iS = s_iS[g];
          float *row = s_p + g * kRow;
          // exp(-inf) = 0 for the positions past the end
          *reinterpret_cast<float4 *>(row + kHalo + 4 * tid) =
              make_float4(__expf(z[g].x - M) * iS, __expf(z[g].y - M) * iS, __expf(z[g].z - M) * iS,
                          __expf(z[g].w - M) * iS);
          if (tid < 2 * kHalo) row[side ? kHalo + kSelTile + hj : hj] = __expf(zh[g] - M) * iS;
        }
      }
    }
    __syncthreads();
    float sc4[4];
    if (half <= 4) {
      // this thread's 4 positions and up to 4 neighbours on each side, from three aligned vector reads
#pragma unroll
      for (int j = 0; j < 4; ++j) sc4[j] = 0.f;
      for (int g = 0; g < p.G; ++g) {
        const float4 *c4 = reinterpret_cast<const float4 *>(s_p + g * kRow + kHalo + 4 * tid - 4);
        const float4 a = c4[0], bq = c4[1], cq = c4[2];
        const float f[12] = {a.x, a.y, a.z, a.w, bq.x, bq.y, bq.z, bq.w, cq.x, cq.y, cq.z, cq.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float v;
          if (p.pool_mode == S4R_POOL_MAX) {
            v = f[4 + j];
#pragma unroll
            for (int d = 1; d <= 4; ++d)
              if (d <= half) v = fmaxf(v, fmaxf(f[4 + j - d], f[4 + j + d]));
          } else {
            v = 0.f;
#pragma unroll
            for (int d = -4; d <= 4; ++d)
              if (d >= -half && d <= half) v += f[4 + j + d];
            v *= inv_kappa;
          }
          sc4[j] = (p.group_mode == S4R_GROUP_MEAN) ? sc4[j] + v : fmaxf(sc4[j], v);
        }
      }
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float agg = 0.f;
        for (int g = 0; g < p.G; ++g) {
          const float *c = s_p + g * kRow + kHalo + 4 * tid + j;
          float v;
          if (p.pool_mode == S4R_POOL_MAX) {
            v = c[0];
            for (int d = 1; d <= half; ++d) v = fmaxf(v, fmaxf(c[-d], c[d]));
          } else {
            v = c[-half];
            for (int d = -half + 1; d <= half; ++d) v += c[d];
            v *= inv_kappa;
          }
          agg = (p.group_mode == S4R_GROUP_MEAN) ? agg + v : fmaxf(agg, v);
        }
        sc4[j] = agg;
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int l = l0 + 4 * tid + j;
      const float agg = (p.group_mode == S4R_GROUP_MEAN) ? sc4[j] * inv_G : sc4[j];
      if (l < end) score[l - begin] = agg;
      // histogram of the top 11 bits; lanes that hit the same bin send one atomic (scores cluster in few bins)
      const bool valid = l < end && l < n_cand;
      const unsigned bin = valid ? (__float_as_uint(agg) >> 21) : 0xffffffffu;
      const unsigned peers = __match_any_sync(0xffffffffu, bin);
      if (valid && lane == __ffs(peers) - 1) atomicAdd(&s_hist[bin], (unsigned)__popc(peers));
    }
    __syncthreads();
  }

  // ---- radix select of the k_eff-th largest candidate score
  const int c_end = min(end, n_cand);
  unsigned k_rem = (unsigned)k_eff, above;
  const unsigned bin1 = find_bin(cluster, s_hist, s_tot, s_warp, s_bc, 2048, k_rem, &above);
  k_rem -= above;
  for (int i = tid; i < 2048; i += kSelThreads) s_hist[i] = 0;
  __syncthreads();
  for (int l = begin + tid; l < c_end; l += kSelThreads) {
    unsigned v = __float_as_uint(score[l - begin]);
    if ((v >> 21) == bin1) atomicAdd(&s_hist[(v >> 10) & 0x7ffu], 1u);
  }
  const unsigned bin2 = find_bin(cluster, s_hist, s_tot, s_warp, s_bc, 2048, k_rem, &above);
  k_rem -= above;
  const unsigned pre2 = (bin1 << 11) | bin2;
  for (int i = tid; i < 2048; i += kSelThreads) s_hist[i] = 0;
  __syncthreads();
  for (int l = begin + tid; l < c_end; l += kSelThreads) {
    unsigned v = __float_as_uint(score[l - begin]);
    if ((v >> 10) == pre2) atomicAdd(&s_hist[v & 0x3ffu], 1u);
  }
  const unsigned bin3 = find_bin(cluster, s_hist, s_tot, s_warp, s_bc, 1024, k_rem, &above);
  k_rem -= above;  // how many candidates equal to the threshold are taken (lowest indices first)
  const unsigned tau = (pre2 << 10) | bin3;

  // ---- each warp owns a contiguous chunk of the slice: count, exchange, then write in index order
  int chunk = (max(c_end - begin, 0) + 31) / 32;
  chunk = (chunk + 31) & ~31;
  const int wbeg = min(c_end, begin + warp * chunk), wend = min(c_end, wbeg + chunk);
  {
    unsigned ngt = 0, neq = 0;
    for (int l = wbeg + lane; l < wend; l += 32) {
      const unsigned v = __float_as_uint(score[l - begin]);
      ngt += v > tau;
      neq += v == tau;
    }
    ngt = __reduce_add_sync(0xffffffffu, ngt);
    neq = __reduce_add_sync(0xffffffffu, neq);
    if (lane == 0) {
      s_wcnt[warp][0] = ngt;
      s_wcnt[warp][1] = neq;
    }
  }
  __syncthreads();
  if (warp == 0) {
    const unsigned a = __reduce_add_sync(0xffffffffu, s_wcnt[lane][0]);
    const unsigned e = __reduce_add_sync(0xffffffffu, s_wcnt[lane][1]);
    // push this CTA's totals into the slot `rank` of every higher-ranked CTA
    if (lane > rank && lane < CL) {
      unsigned(*dst)[2] = reinterpret_cast<unsigned(*)[2]>(cluster.map_shared_rank(&s_cnts[0][0], lane));
      dst[rank][0] = a;
      dst[rank][1] = e;
    }
  }
  cluster.sync();
  unsigned gt_before = 0, eq_before = 0;
  for (int rk = 0; rk < rank; ++rk) {
    gt_before += s_cnts[rk][0];
    eq_before += s_cnts[rk][1];
  }
  // prefix over the warps of this CTA (every warp computes it redundantly; lane i stands for warp i)
  unsigned my_gt = s_wcnt[lane][0], my_eq = s_wcnt[lane][1];
  unsigned eq_inc = my_eq;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    unsigned t = __shfl_up_sync(0xffffffffu, eq_inc, o);
    if (lane >= o) eq_inc += t;
  }
  const unsigned eq_pre = eq_before + eq_inc - my_eq;                  // equal elements before warp `lane`
  const unsigned taken = eq_pre >= k_rem ? 0u : min(my_eq, k_rem - eq_pre);
  unsigned sel_inc = my_gt + taken;
  const unsigned my_sel = sel_inc;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    unsigned t = __shfl_up_sync(0xffffffffu, sel_inc, o);
    if (lane >= o) sel_inc += t;
  }
  const unsigned cta_base = gt_before + min(eq_before, k_rem);
  unsigned out_pos = __shfl_sync(0xffffffffu, cta_base + sel_inc - my_sel, warp);
  unsigned eq_seen = __shfl_sync(0xffffffffu, eq_pre, warp);
  const unsigned lt_mask = (1u << lane) - 1u;
  for (int l0 = wbeg; l0 < wend; l0 += 32) {
    const int l = l0 + lane;
    const bool in = l < wend;
    const unsigned v = in ? __float_as_uint(score[l - begin]) : 0u;
    const bool is_eq = in && v == tau;
    const unsigned eq_mask = __ballot_sync(0xffffffffu, is_eq);
    const bool take = in && (v > tau || (is_eq && eq_seen + __popc(eq_mask & lt_mask) < k_rem));
    const unsigned take_mask = __ballot_sync(0xffffffffu, take);
    if (take) out_idx[out_pos + __popc(take_mask & lt_mask)] = l;
    out_pos += __popc(take_mask);
    eq_seen += __popc(eq_mask);
  }
  // no remote access follows the exchange of the counts, so CTAs may leave independently
}

}  // namespace

cudaError_t launch_select(const StepArgs &a) {
  SelParams p;
  p.Z = (const float *)(a.ws + a.plan.off_z);
  p.part = (const float2 *)(a.ws + a.plan.off_part);
  p.coef_len = a.coef_len;
  p.score = (float *)(a.ws + a.plan.off_score);
  p.sel_idx = a.sel_idx;
  p.sel_count = a.sel_count;
  p.G = a.ly.G;
  p.n_parts = a.plan.n_parts;
  p.window = a.window;
  p.top_k = a.top_k;
  p.kappa = a.kappa;
  p.pool_mode = a.pool_mode;
  p.group_mode = a.group_mode;
  p.max_len = a.plan.max_len;
  p.z_stride = a.plan.z_stride;
  p.dev_status = a.dev_status;
  const size_t smem = sizeof(float) * ((size_t)kSliceCap + (size_t)a.ly.G * (kSelTile + 2 * kHalo));
  static size_t smem_set = 0;
  if (smem > smem_set) {
    cudaError_t e = cudaFuncSetAttribute(k_select, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    smem_set = smem;
  }
  int cluster = a.plan.cluster;
  if (cluster > 8) {  // 16 CTAs per cluster is beyond the portable size: opt in once and check that it can be placed
    static int ok16 = -1;
    if (ok16 < 0) {
      ok16 = 0;
      if (cudaFuncSetAttribute(k_select, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
        cudaLaunchConfig_t probe = {};
        probe.gridDim = dim3(16, 1);
        probe.blockDim = dim3(kSelThreads);
        probe.dynamicSmemBytes = smem;
        cudaLaunchAttribute pa[1];
        pa[0].id = cudaLaunchAttributeClusterDimension;
        pa[0].val.clusterDim.x = 16;
        pa[0].val.clusterDim.y = 1;
        pa[0].val.clusterDim.z = 1;
        probe.attrs = pa;
        probe.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, k_select, &probe) == cudaSuccess && n >= 1) ok16 = 1;
      }
      (void)cudaGetLastError();
    }
    if (!ok16) cluster = 8;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(cluster, a.ly.B);
  cfg.blockDim = dim3(kSelThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = a.stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, k_select, p);
  if (e != cudaSuccess) return e;
  ++launch_counter();
  return cudaGetLastError();
}

}  // namespace s4r
