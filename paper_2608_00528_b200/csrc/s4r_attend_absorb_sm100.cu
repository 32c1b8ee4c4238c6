// Sparse reconstruction + attention (Eq. 16-18) for bf16 caches on sm_100a, value side absorbed:
//   O = P V^ = P (C^V[rows] (B^V)^T) = (P C^V[rows]) (B^V)^T.
// The keys are reconstructed exactly as Eq. 16 says (they must be: RoPE sits between the reconstruction and
// the dot product).  For the values the same product is evaluated in the other order: each tile contracts its
// probabilities with the gathered value coefficients on the tensor cores, U[g, :] = sum_t p[t, g] C^V[row_t, :],
// and the multiplication by the value basis happens once per (sequence, head) after the tiles have been
// merged (k_merge_absorb).  Same result up to fp32 rounding order; it removes the value-basis stream, the
// V^ accumulator read-back and the per-token P.V^ loop from this kernel.
//
// One CTA owns a tile of 128 selected rows and a range of KV heads.  Gathered rows sit in 128-byte-swizzled
// shared memory; per head
//   K^[tokens x d_h] = C^K[rows] (B^K slice)^T   tcgen05.mma, basis slice streamed through a TMA ring
//   logits, tile softmax                         16 epilogue warps, RoPE angles held in registers
//   U[2G x r_v]      = [P_hi; P_lo]^T C^V[rows]  tcgen05.mma, probabilities as two bf16 terms (hi + lo)
// Warp 0 = TMA producer, warp 1 = MMA issuer, warps 2-17 = epilogue.
#include "s4r_internal.h"
#include "s4r_sm100.cuh"

namespace s4r {

using namespace sm100;

void fill_inv_freq(double *dst, int head_dim, float theta);

namespace {

constexpr int kTok = 128;
constexpr int kDh = 128;
constexpr int kRing = 3;
constexpr int kBlkBytes = 128 * 128;
constexpr int kEpiWarps = 16;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kThreads = 64 + kEpiThreads;

struct AbsorbParams {
  const __nv_bfloat16 *q, *coef_k, *coef_v;
  const int32_t *coef_len, *sel_idx, *sel_count;
  float *part_u;    // [B][Hq][tiles][2 (hi, lo part of P)][rv]
  float2 *part_ms;  // [B][Hq][tiles]
  int Hq, Hkv, G, D, rk, rv, s, n_tiles, sel_stride, nkv;
  int64_t cap, max_len;
  float theta;
  int32_t *dev_status;
  double inv_freq[64];
};

__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }
__device__ __forceinline__ float2 bcast2(float v) { return make_float2(v, v); }
__device__ __forceinline__ void cp_async16_zfill(void *dst, const void *src, bool valid) {
  const int n = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(n) : "memory");
}

__global__ void __launch_bounds__(kThreads, 1) k_attend_absorb(const __grid_constant__ CUtensorMap tmap_bk,
                                                               const __grid_constant__ AbsorbParams p) {
  grid_dependency_sync();
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int kbk = p.rk >> 6, kbv = p.rv >> 6, G = p.G;
  uint8_t *ck = smem;                                   // [kbk][128 tokens][128 B]   A of the K^ product
  uint8_t *cv = ck + (size_t)kbk * kBlkBytes;           // [kbv][128 tokens][128 B]   B (N-contiguous) of P C^V
  uint8_t *ring = cv + (size_t)kbv * kBlkBytes;         // [kRing][128 d][128 B]      key-basis blocks
  uint8_t *pop = ring + (size_t)kRing * kBlkBytes;      // [2][128 rows][128 B]       A of P C^V: rows g / G+g = hi / lo
  float *qs = reinterpret_cast<float *>(pop + 2 * kBlkBytes);   // [128 cols][8]
  float *xch = qs + kDh * kMaxGroup;                             // [4 quarters][G][128]
  uint64_t *bars = reinterpret_cast<uint64_t *>(xch + 4 * G * 128);
  uint64_t *full = bars, *empty = bars + kRing;
  uint64_t *k_full = bars + 2 * kRing, *k_empty = k_full + 2;
  uint64_t *p_ready = k_empty + 2, *u_full = p_ready + 1, *u_empty = u_full + 1;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(u_empty + 1);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  int *rows = reinterpret_cast<int *>(tmem_slot + 2);   // [128]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile = blockIdx.x, kv0 = blockIdx.y * p.nkv, b = blockIdx.z;
  const int count = min(p.sel_count[b], p.sel_stride);
  const int t0 = tile * kTok;
  if (t0 >= count) return;  // uniform over the CTA
  const int nt = min(kTok, count - t0);
  int L = p.coef_len[b];
  L = L < 0 ? 0 : (L > p.max_len ? (int)p.max_len : L);

  if (tid == 0) {
    for (int i = 0; i < kRing; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&k_full[i], 1);
      mbar_init(&k_empty[i], kEpiWarps);
    }
    mbar_init(p_ready, 1);
    mbar_init(u_full, 1);
    mbar_init(u_empty, 4);  // the four warps of lane quadrant 0 read U
    *abort_flag = 0;
    mbar_fence_init();
    prefetch_tmap(&tmap_bk);
  }
  if (warp == 1) tmem_alloc(tmem_slot, 512);
  if (tid < kTok) {
    int rix = (tid < nt) ? p.sel_idx[(size_t)b * p.sel_stride + t0 + tid] : -1;
    rows[tid] = rix < 0 ? -1 : min(rix, max(L - 1, 0));
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp != 0) {
    // ---- gather the selected coefficient rows (asynchronous 16-byte pieces, all in flight at once; rows past
    //      the tile's end are zero) and clear the probability operand, while the producer fills the ring
    constexpr int kWorkers = kThreads - 32;
    const int wt = tid - 32;
    const int cpr_k = p.rk >> 3, cpr_v = p.rv >> 3;
    const __nv_bfloat16 *ckb = p.coef_k + (size_t)b * p.cap * p.rk;
    const __nv_bfloat16 *cvb = p.coef_v + (size_t)b * p.cap * p.rv;
    for (int i = wt; i < kTok * cpr_k; i += kWorkers) {
      const int t = i / cpr_k, c = i - t * cpr_k, rix = rows[t];
      cp_async16_zfill(ck + (size_t)(c >> 3) * kBlkBytes + sw128_offset(t, (c & 7) * 8),
                       reinterpret_cast<const uint4 *>(ckb + (size_t)max(rix, 0) * p.rk) + c, rix >= 0);
    }
    for (int i = wt; i < kTok * cpr_v; i += kWorkers) {
      const int t = i / cpr_v, c = i - t * cpr_v, rix = rows[t];
      cp_async16_zfill(cv + (size_t)(c >> 3) * kBlkBytes + sw128_offset(t, (c & 7) * 8),
                       reinterpret_cast<const uint4 *>(cvb + (size_t)max(rix, 0) * p.rv) + c, rix >= 0);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    for (int i = wt; i < 2 * kBlkBytes / 16; i += kWorkers) reinterpret_cast<uint4 *>(pop)[i] = make_uint4(0, 0, 0, 0);
  }

  if (warp == 0) {
    // ---------------- TMA producer: key-basis slices in 64-column blocks ----------------
    if (lane == 0) {
      int it = 0, issued = 0;
      bool ok = true;
      for (int h = 0; h < p.nkv && ok; ++h) {
        const int y = b * p.D + (kv0 + h) * kDh;
        for (int blk = 0; blk < kbk; ++blk, ++it) {
          const int slot = it % kRing;
          if (!mbar_wait(&empty[slot], ((uint32_t)(it / kRing) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
          mbar_expect_tx(&full[slot], kBlkBytes);
          tma_load_2d(ring + (size_t)slot * kBlkBytes, &tmap_bk, blk * 64, y, &full[slot]);
          issued = it + 1;
        }
      }
      if (*abort_flag) {
        for (int i = max(0, issued - kRing); i < issued; ++i) {
          const unsigned long long t_0 = global_ns();
          while (!mbar_try_wait(&full[i % kRing], (uint32_t)(i / kRing) & 1u))
            if (global_ns() - t_0 > kWaitLimitNs) break;
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    fence_proxy_async_smem();
    asm volatile("bar.sync 2, %0;" ::"n"(kThreads - 32) : "memory");  // tiles gathered, operand cleared
    if (lane == 0) {
      const uint32_t idesc_k = umma_idesc_bf16(128, 128);
      const uint32_t idesc_u = umma_idesc_bf16(128, p.rv) | (1u << 16);  // B operand N-contiguous
      const uint64_t ck_desc = umma_desc_sw128(smem_u32(ck));
      const uint64_t cv_desc = umma_desc_mn_sw128(smem_u32(cv), kBlkBytes);
      const uint64_t pop_desc = umma_desc_sw128(smem_u32(pop));
      int it = 0;
      bool ok = true;
      auto issue_k = [&](int h) {
        const int buf = h & 1;
        if (!mbar_wait(&k_empty[buf], ((uint32_t)(h >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; return; }
        tc_fence_after();
        for (int blk = 0; blk < kbk; ++blk, ++it) {
          const int slot = it % kRing;
          if (!mbar_wait(&full[slot], (uint32_t)(it / kRing) & 1u, abort_flag)) { ok = false; return; }
          tc_fence_after();
          const uint64_t bs_desc = umma_desc_sw128(smem_u32(ring + (size_t)slot * kBlkBytes));
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)
            umma_bf16(tmem_base + (uint32_t)buf * 128, ck_desc + (uint64_t)((blk * kBlkBytes + k4 * 32) >> 4),
                      bs_desc + (uint64_t)((k4 * 32) >> 4), idesc_k, (blk | k4) != 0);
          umma_commit(&empty[slot]);
        }
        umma_commit(&k_full[buf]);
      };
      issue_k(0);
      for (int h = 0; h < p.nkv && ok; ++h) {
        if (h + 1 < p.nkv) issue_k(h + 1);  // the key product runs one head ahead of the epilogue
        if (!ok) break;
        // U = [P_hi; P_lo]^T C^V over the 128 tokens of the tile (8 steps of 16 tokens)
        if (!mbar_wait(p_ready, (uint32_t)h & 1u, abort_flag)) break;
        if (!mbar_wait(u_empty, ((uint32_t)h & 1u) ^ 1u, abort_flag)) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          umma_bf16(tmem_base + 256u, pop_desc + (uint64_t)(((kk >> 2) * kBlkBytes + (kk & 3) * 32) >> 4),
                    cv_desc + (uint64_t)((kk * 2048) >> 4), idesc_u, kk != 0);
        umma_commit(u_full);
      }
    }
  } else {
    // ---------------- epilogue: 16 warps; warps e, e+4, e+8, e+12 share a TMEM lane quadrant ----------------
    const int e = warp - 2, et = tid - 64;
    const int quad = warp & 3, qt = e >> 2;
    const int lane_row = quad * 32 + lane;   // token owned by this thread
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const int npair = (G + 1) >> 1;
    const bool rope = p.theta > 0.f;
    // RoPE angles of this thread's token for its 16 pairs, kept in registers for all heads
    // (sin, cos) packed as two 16-bit fixed-point numbers (absolute error 1.5e-5, far below bf16 resolution)
    uint32_t sc[16];
    {
      const int rix = rows[lane_row];
#pragma unroll
      for (int ii = 0; ii < 16; ++ii) {
        float sn = 0.f, cs = 1.f;
        if (rope && rix >= 0) rope_sincos(p.s + rix, p.inv_freq[qt * 16 + ii], sn, cs);
        sc[ii] = ((uint32_t)__float2int_rn(sn * 32767.f) & 0xffffu) | ((uint32_t)__float2int_rn(cs * 32767.f) << 16);
      }
    }
    // q' = RoPE(q) / sqrt(d_h), laid out [col][g]; this thread prepares column qc for the heads g = qg0, qg0 + 4.
    // The raw values of the next KV head are fetched one head ahead.
    const int qc = et & 127, qg0 = et >> 7;
    float q_sn = 0.f, q_cs = 1.f;
    if (rope) rope_sincos(p.s + L - 1, p.inv_freq[qc & 63], q_sn, q_cs);
    const float q_scale = rsqrtf((float)kDh);
    float q_raw[2][2];  // [g slot][own, partner]
    auto fetch_q = [&](int h) {
#pragma unroll
      for (int sl = 0; sl < 2; ++sl) {
        const int g = qg0 + 4 * sl;
        q_raw[sl][0] = q_raw[sl][1] = 0.f;
        if (g < G && h < p.nkv) {
          const __nv_bfloat16 *qp = p.q + ((size_t)b * p.Hq + (size_t)(kv0 + h) * G + g) * kDh;
          q_raw[sl][0] = __bfloat162float(qp[qc]);
          q_raw[sl][1] = __bfloat162float(qp[qc ^ 64]);
        }
      }
    };
    auto store_q = [&]() {
#pragma unroll
      for (int sl = 0; sl < 2; ++sl) {
        float v = q_raw[sl][0];
        if (rope) v = (qc < 64) ? v * q_cs - q_raw[sl][1] * q_sn : v * q_cs + q_raw[sl][1] * q_sn;
        qs[qc * kMaxGroup + qg0 + 4 * sl] = v * q_scale;
      }
    };
    // U of one head: TMEM lanes 0..G-1 hold the hi part, G..2G-1 the lo part; the four warps of quadrant 0 split
    // the columns and store both parts (k_merge_absorb adds them)
    auto read_u = [&](int h, bool ok_in) -> bool {
      bool ok2 = ok_in;
      if (ok2) ok2 = mbar_wait(u_full, (uint32_t)h & 1u, abort_flag);
      ok2 = __all_sync(0xffffffffu, ok2);
      tc_fence_after();
      if (ok2) {
        const int cper = p.rv >> 2;  // columns per warp, a multiple of 16
        const int part = lane < G ? 0 : 1, g = lane < G ? lane : lane - G;
        float *dst = p.part_u + ((((size_t)b * p.Hq + (size_t)(kv0 + h) * G + min(g, G - 1)) * p.n_tiles + tile) * 2 + part) * p.rv;
        for (int c0 = qt * cper; c0 < (qt + 1) * cper; c0 += 16) {
          uint32_t v[16];
          tmem_ld16(tmem_base + 256u + (uint32_t)c0, v);
          tmem_ld_wait();
          if (lane < 2 * G) {
#pragma unroll
            for (int j = 0; j < 16; j += 4)
              *reinterpret_cast<float4 *>(dst + c0 + j) = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]),
                                                                      __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(u_empty);
      }
      return ok2;
    };
    fetch_q(0);
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    fence_proxy_async_smem();
    store_q();
    fetch_q(1);
    asm volatile("bar.sync 2, %0;" ::"n"(kThreads - 32) : "memory");  // tiles gathered, operand cleared, q' of head 0 set
    bool ok = true;  // warp-uniform; after a failed wait the loop keeps its shape but touches tensor memory no more
    for (int h = 0; h < p.nkv; ++h) {
      const int kv = kv0 + h, buf = h & 1;
      const uint32_t aph = (uint32_t)(h >> 1) & 1u;
      // ---- K^ row of this thread's token: pairs [16*qt, +16)
      if (ok) ok = mbar_wait(&k_full[buf], aph, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      float2 lg[4];
#pragma unroll
      for (int gp = 0; gp < 4; ++gp) lg[gp] = make_float2(0.f, 0.f);
      if (ok) {
        uint32_t ka[16], kb[16];
        const uint32_t base = tmem_base + (uint32_t)buf * 128 + lane_addr + (uint32_t)qt * 16;
        tmem_ld16(base, ka);
        tmem_ld16(base + 64, kb);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&k_empty[buf]);
#pragma unroll
        for (int ii = 0; ii < 16; ++ii) {
          const int i = qt * 16 + ii;
          float2 k12 = make_float2(__uint_as_float(ka[ii]), __uint_as_float(kb[ii]));
          if (rope) {
            const float sn = (float)(short)(sc[ii] & 0xffffu) * (1.f / 32767.f);
            const float cs = (float)((int)sc[ii] >> 16) * (1.f / 32767.f);
            k12 = __ffma2_rn(make_float2(-k12.y, k12.x), bcast2(sn), __fmul2_rn(k12, bcast2(cs)));
          }
          const float2 k1 = bcast2(k12.x), k2 = bcast2(k12.y);
          const float4 qa = *reinterpret_cast<const float4 *>(qs + i * kMaxGroup);
          const float4 qb = *reinterpret_cast<const float4 *>(qs + (i + 64) * kMaxGroup);
          lg[0] = __ffma2_rn(make_float2(qa.x, qa.y), k1, __ffma2_rn(make_float2(qb.x, qb.y), k2, lg[0]));
          lg[1] = __ffma2_rn(make_float2(qa.z, qa.w), k1, __ffma2_rn(make_float2(qb.z, qb.w), k2, lg[1]));
          if (npair > 2) {
            const float4 qc4 = *reinterpret_cast<const float4 *>(qs + i * kMaxGroup + 4);
            const float4 qd4 = *reinterpret_cast<const float4 *>(qs + (i + 64) * kMaxGroup + 4);
            lg[2] = __ffma2_rn(make_float2(qc4.x, qc4.y), k1, __ffma2_rn(make_float2(qd4.x, qd4.y), k2, lg[2]));
            lg[3] = __ffma2_rn(make_float2(qc4.z, qc4.w), k1, __ffma2_rn(make_float2(qd4.z, qd4.w), k2, lg[3]));
          }
        }
      }
#pragma unroll
      for (int gp = 0; gp < 4; ++gp) {
        if (2 * gp < G) xch[(qt * G + 2 * gp) * 128 + lane_row] = lg[gp].x;
        if (2 * gp + 1 < G) xch[(qt * G + 2 * gp + 1) * 128 + lane_row] = lg[gp].y;
      }
      epi_sync();  // logits exchanged; q' of this head is no longer read
      // ---- tile softmax by warp e for head g = e; probabilities go into the MMA operand as hi + lo bf16
      if (e < G) {
        float l4[4], m = -INFINITY;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int t = u * 32 + lane;
          l4[u] = (t < nt) ? (xch[e * 128 + t] + xch[(G + e) * 128 + t]) + (xch[(2 * G + e) * 128 + t] + xch[(3 * G + e) * 128 + t])
                           : -INFINITY;
          m = fmaxf(m, l4[u]);
        }
        m = warp_max(m);
        float ssum = 0.f;
        // the previous head's P C^V must have read the operand before it is overwritten
        if (ok && h > 0) ok = mbar_wait(u_full, (uint32_t)(h - 1) & 1u, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int t = u * 32 + lane;
          const float pe = (l4[u] == -INFINITY) ? 0.f : __expf(l4[u] - m);
          ssum += pe;
          const __nv_bfloat16 hi = __float2bfloat16_rn(pe);
          const __nv_bfloat16 lo = __float2bfloat16_rn(pe - __bfloat162float(hi));
          uint8_t *blk = pop + (size_t)(t >> 6) * kBlkBytes;
          *reinterpret_cast<__nv_bfloat16 *>(blk + sw128_offset(e, t & 63)) = hi;
          *reinterpret_cast<__nv_bfloat16 *>(blk + sw128_offset(G + e, t & 63)) = lo;
        }
        ssum = warp_sum(ssum);
        if (lane == 0) p.part_ms[((size_t)b * p.Hq + (size_t)kv * G + e) * p.n_tiles + tile] = make_float2(m, ssum);
        fence_proxy_async_smem();
      }
      store_q();       // q' of the next head
      fetch_q(h + 2);  // raw values two heads ahead
      if (quad == 0 && h > 0) ok = read_u(h - 1, ok);  // the previous head's U, whose MMA ran during this head's K loop
      epi_sync();
      if (et == 0) mbar_arrive(p_ready);
    }
    if (quad == 0) ok = read_u(p.nkv - 1, ok);
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *abort_flag && p.dev_status) atomicOr(p.dev_status, S4R_DEV_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// ------------------------------------------------------------------------------------------------------------
// Merge for the absorbed value path: joins the tiles' (max, sum, U) with the sinks and applies the value basis:
//   out[d] = ( sum_j (sum_t w_t U_t[j]) B^V[kv*d_h + d][j] + sum_sinks w_s v_s[d] ) / (sum_t w_t s_t + sum_s w_s)
// grid (Hq, B), block 128 threads (thread = output channel d).
// ------------------------------------------------------------------------------------------------------------
struct MergeAbsorbParams {
  const __nv_bfloat16 *q, *sink_k, *sink_v, *basis_v;
  const int32_t *coef_len, *sel_count;
  const float *part_u;
  const float2 *part_ms;
  void *out;
  int out_dtype, Hq, G, D, rv, s, n_tiles, sel_stride;
  int64_t max_len;
  float theta;
  double inv_freq[64];
};

__device__ __forceinline__ void cp_async16(void *dst, const void *src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async8(void *dst, const void *src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}

constexpr int kMgTiles = 32;

__global__ void __launch_bounds__(128) k_merge_absorb(const __grid_constant__ MergeAbsorbParams p) {
  grid_dependency_sync();
  extern __shared__ __align__(16) uint8_t msm[];
  const int h = blockIdx.x, b = blockIdx.y, i = threadIdx.x;
  const int kv = h / p.G, lane = i & 31, warp = i >> 5;
  const int rvp = p.rv + 8;  // padded row of the staged basis slice (bank spread)
  __nv_bfloat16 *bv_s = reinterpret_cast<__nv_bfloat16 *>(msm);                    // [128][rv + 8]
  __nv_bfloat16 *q_s = bv_s + (size_t)kDh * rvp;                                    // [128]
  __nv_bfloat16 *sk_s = q_s + kDh;                                                  // [s][128]
  __nv_bfloat16 *sv_s = sk_s + (size_t)p.s * kDh;                                   // [s][128]
  float *pu_s = reinterpret_cast<float *>(sv_s + (size_t)p.s * kDh);                // [kMgTiles][2][rv]
  float2 *ms_s = reinterpret_cast<float2 *>(pu_s + (size_t)kMgTiles * 2 * p.rv);    // [kMgTiles]
  float *ut_s = reinterpret_cast<float *>(ms_s + kMgTiles);                         // [rv]
  float *red_s = ut_s + p.rv;                                                       // [4][64]
  float *slog_s = red_s + 4 * 64;                                                   // [64]

  int L = p.coef_len[b];
  L = L < 0 ? 0 : ((int64_t)L > p.max_len ? (int)p.max_len : L);
  const int count = min(p.sel_count[b], p.sel_stride);
  const int tiles = (count + kTok - 1) / kTok;
  const float2 *ms = p.part_ms + ((size_t)b * p.Hq + h) * p.n_tiles;
  const float *pu = p.part_u + ((size_t)b * p.Hq + h) * p.n_tiles * 2 * p.rv;
  // ---- one wave of asynchronous copies
  {
    const int cpr = p.rv >> 3;
    const __nv_bfloat16 *bvp = p.basis_v + ((size_t)b * p.D + (size_t)kv * kDh) * p.rv;
    for (int c = i; c < kDh * cpr; c += 128) {
      const int d = c / cpr, cc = c - d * cpr;
      cp_async16(bv_s + (size_t)d * rvp + cc * 8, bvp + (size_t)d * p.rv + cc * 8);
    }
    const __nv_bfloat16 *qp = p.q + ((size_t)b * p.Hq + h) * kDh;
    if (i < 16) cp_async16(q_s + i * 8, qp + i * 8);
    for (int c = i; c < p.s * 16; c += 128) {
      const int sj = c >> 4, cc = c & 15;
      const size_t off = ((size_t)b * p.s + sj) * p.D + (size_t)kv * kDh + cc * 8;
      cp_async16(sk_s + sj * kDh + cc * 8, p.sink_k + off);
      cp_async16(sv_s + sj * kDh + cc * 8, p.sink_v + off);
    }
    const int nt0 = min(tiles, kMgTiles);
    if (i < nt0) cp_async8(ms_s + i, ms + i);
    for (int c = i; c < nt0 * (p.rv >> 1); c += 128) cp_async16(pu_s + c * 4, pu + c * 4);
  }
  float M = -INFINITY;
  if (tiles > kMgTiles) {
    for (int t = i; t < tiles; t += 128) M = fmaxf(M, ms[t].x);
    M = warp_max(M);
    if (lane == 0) red_s[warp] = M;
  }
  asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
  __syncthreads();
  if (tiles > kMgTiles) {
    M = fmaxf(fmaxf(red_s[0], red_s[1]), fmaxf(red_s[2], red_s[3]));
  } else {
    for (int t = 0; t < tiles; ++t) M = fmaxf(M, ms_s[t].x);
  }
  __syncthreads();
  // ---- rotated, scaled query channel and the sink logits
  const bool rope = p.theta > 0.f;
  const int partner = i < 64 ? i + 64 : i - 64;
  const double inv_freq = p.inv_freq[i & 63];
  float qi = __bfloat162float(q_s[i]);
  if (rope) {
    const float o = __bfloat162float(q_s[partner]);
    float sn, cs;
    rope_sincos(p.s + L - 1, inv_freq, sn, cs);
    qi = i < 64 ? qi * cs - o * sn : qi * cs + o * sn;
  }
  qi *= rsqrtf((float)kDh);
  for (int sj = 0; sj < p.s; ++sj) {
    float v = __bfloat162float(sk_s[sj * kDh + i]);
    if (rope) {
      const float o = __bfloat162float(sk_s[sj * kDh + partner]);
      float sn, cs;
      rope_sincos(sj, inv_freq, sn, cs);
      v = i < 64 ? v * cs - o * sn : v * cs + o * sn;
    }
    const float d = warp_sum(qi * v);
    if (lane == 0) red_s[warp * 64 + sj] = d;
  }
  __syncthreads();
  if (i < p.s) slog_s[i] = (red_s[i] + red_s[64 + i]) + (red_s[128 + i] + red_s[192 + i]);
  __syncthreads();
  for (int sj = 0; sj < p.s; ++sj) M = fmaxf(M, slog_s[sj]);
  // ---- weighted sum of the tiles' U (thread j handles coefficient columns j, j + 128, ...)
  float den = 0.f;
  float ut[4] = {0.f, 0.f, 0.f, 0.f};  // rv <= 512
  for (int t0 = 0; t0 < tiles; t0 += kMgTiles) {
    const int nt = min(kMgTiles, tiles - t0);
    if (t0 > 0) {
      __syncthreads();
      if (i < nt) cp_async8(ms_s + i, ms + t0 + i);
      for (int c = i; c < nt * (p.rv >> 1); c += 128) cp_async16(pu_s + c * 4, pu + (size_t)t0 * 2 * p.rv + c * 4);
      asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
      __syncthreads();
    }
    for (int t = 0; t < nt; ++t) {
      const float2 v = ms_s[t];
      const float w = v.y > 0.f ? __expf(v.x - M) : 0.f;
      den = fmaf(v.y, w, den);
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        const int j = i + 128 * jj;
        if (j < p.rv) ut[jj] = fmaf(pu_s[t * 2 * p.rv + j] + pu_s[t * 2 * p.rv + p.rv + j], w, ut[jj]);
      }
    }
  }
#pragma unroll
  for (int jj = 0; jj < 4; ++jj) {
    const int j = i + 128 * jj;
    if (j < p.rv) ut_s[j] = ut[jj];
  }
  __syncthreads();
  // ---- out[d] = <u_tot, B^V[kv*d_h + d]> + sinks
  float num = 0.f;
  {
    const __nv_bfloat16 *row = bv_s + (size_t)i * rvp;
    for (int j = 0; j < p.rv; j += 8) {
      const uint4 raw = *reinterpret_cast<const uint4 *>(row + j);
      const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
      const float4 u0 = *reinterpret_cast<const float4 *>(ut_s + j), u1 = *reinterpret_cast<const float4 *>(ut_s + j + 4);
      num = fmaf(__uint_as_float(w[0] << 16), u0.x, num);
      num = fmaf(__uint_as_float(w[0] & 0xffff0000u), u0.y, num);
      num = fmaf(__uint_as_float(w[1] << 16), u0.z, num);
      num = fmaf(__uint_as_float(w[1] & 0xffff0000u), u0.w, num);
      num = fmaf(__uint_as_float(w[2] << 16), u1.x, num);
      num = fmaf(__uint_as_float(w[2] & 0xffff0000u), u1.y, num);
      num = fmaf(__uint_as_float(w[3] << 16), u1.z, num);
      num = fmaf(__uint_as_float(w[3] & 0xffff0000u), u1.w, num);
    }
  }
  for (int sj = 0; sj < p.s; ++sj) {
    const float w = __expf(slog_s[sj] - M);
    den += w;
    num = fmaf(__bfloat162float(sv_s[sj * kDh + i]), w, num);
  }
  const float o = (tiles + p.s > 0 && den > 0.f) ? num / den : 0.f;
  const size_t oi = ((size_t)b * p.Hq + h) * kDh + i;
  if (p.out_dtype == S4R_F32)
    ((float *)p.out)[oi] = o;
  else
    ((__nv_bfloat16 *)p.out)[oi] = __float2bfloat16_rn(o);
}

}  // namespace

int att_fast_kvsplit(const Layer &ly, int n_tiles);

cudaError_t launch_attend_absorb(const StepArgs &a) {
  const Layer &ly = a.ly;
  if (a.plan.n_att_tiles == 0) return cudaSuccess;
  CUtensorMap tm_k;
  if (!make_tmap_bf16_2d(&tm_k, a.basis_k, (uint64_t)ly.B * ly.D, (uint64_t)ly.rk, 128)) return cudaErrorInvalidValue;
  AbsorbParams p;
  p.q = (const __nv_bfloat16 *)a.q;
  p.coef_k = (const __nv_bfloat16 *)a.coef_k;
  p.coef_v = (const __nv_bfloat16 *)a.coef_v;
  p.coef_len = a.coef_len;
  p.sel_idx = a.sel_idx;
  p.sel_count = a.sel_count;
  p.part_u = (float *)(a.ws + a.plan.off_att);
  p.part_ms = (float2 *)(a.ws + a.plan.off_att_ms);
  p.Hq = ly.Hq; p.Hkv = ly.Hkv; p.G = ly.G; p.D = ly.D; p.rk = ly.rk; p.rv = ly.rv; p.s = ly.s;
  p.n_tiles = a.plan.n_att_tiles;
  p.sel_stride = a.window + a.top_k;
  const int split = att_fast_kvsplit(ly, p.n_tiles);
  p.nkv = ly.Hkv / split;
  p.cap = ly.cap;
  p.max_len = a.plan.max_len;
  p.theta = a.theta;
  p.dev_status = a.dev_status;
  fill_inv_freq(p.inv_freq, kDh, a.theta);
  const size_t smem = 1024 + (size_t)(ly.rk / 64 + ly.rv / 64 + kRing + 2) * kBlkBytes +
                      sizeof(float) * (kDh * kMaxGroup + 4 * ly.G * 128) + 1024;
  static size_t smem_set = 0;
  if (smem > smem_set) {
    cudaError_t e = cudaFuncSetAttribute(k_attend_absorb, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    smem_set = smem;
  }
  dim3 grid(p.n_tiles, split, ly.B);
  cudaError_t le = launch_chained(k_attend_absorb, grid, dim3(kThreads), smem, a.stream, 1, tm_k, p);
  if (le != cudaSuccess) return le;
  ++launch_counter();
  return cudaGetLastError();
}

cudaError_t launch_merge_absorb(const StepArgs &a) {
  const Layer &ly = a.ly;
  MergeAbsorbParams p;
  p.q = (const __nv_bfloat16 *)a.q;
  p.sink_k = (const __nv_bfloat16 *)a.sink_k;
  p.sink_v = (const __nv_bfloat16 *)a.sink_v;
  p.basis_v = (const __nv_bfloat16 *)a.basis_v;
  p.coef_len = a.coef_len;
  p.sel_count = a.sel_count;
  p.part_u = (const float *)(a.ws + a.plan.off_att);
  p.part_ms = (const float2 *)(a.ws + a.plan.off_att_ms);
  p.out = a.out; p.out_dtype = a.out_dtype; p.Hq = ly.Hq; p.G = ly.G; p.D = ly.D; p.rv = ly.rv; p.s = ly.s;
  p.n_tiles = a.plan.n_att_tiles; p.sel_stride = a.window + a.top_k; p.max_len = a.plan.max_len; p.theta = a.theta;
  fill_inv_freq(p.inv_freq, kDh, a.theta);
  const size_t smem = sizeof(__nv_bfloat16) * ((size_t)kDh * (ly.rv + 8) + kDh + 2 * (size_t)ly.s * kDh) +
                      sizeof(float) * ((size_t)kMgTiles * 2 * ly.rv + ly.rv + 4 * 64 + 64) + sizeof(float2) * kMgTiles + 16;
  static size_t smem_set = 0;
  if (smem > 48 * 1024 && smem > smem_set) {
    cudaError_t e = cudaFuncSetAttribute(k_merge_absorb, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    smem_set = smem;
  }
  dim3 grid(ly.Hq, ly.B);
  cudaError_t le = launch_chained(k_merge_absorb, grid, dim3(128), smem, a.stream, 1, p);
  if (le != cudaSuccess) return le;
  ++launch_counter();
  return cudaGetLastError();
}

}  // namespace s4r
