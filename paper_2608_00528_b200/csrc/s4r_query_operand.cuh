// The attention kernel's logit product wants q' = RoPE(q) / sqrt(d_h) of every KV head as a ready-made
// tensor-core operand (hi + lo bf16 rows, swizzled; layout: query_operand_offset).  The scoring kernels prepare it
// off their critical path: CTA j of a sequence (of cps) prepares heads j, j + cps, ...
#pragma once

#include "s4r_common.cuh"
#include "s4r_sm100.cuh"

namespace s4r {

struct QueryOperandArgs {
  uint8_t *qimg;               // [B][Hkv][kQueryOperandBytes]; nullptr: not wanted
  const __nv_bfloat16 *q;      // [B][Hq][dh], dh = 128
  int Hq, Hkv, Gq, dh, sinks;
  float theta;
  uint64_t rope_turns[64];
};

// Called by `n_threads` threads (index t) of CTA j of sequence b; L = cache rows incl. the current token.
__device__ __forceinline__ void build_query_operand(const QueryOperandArgs &p, int b, int j, int cps, int L, int t,
                                                    int n_threads) {
  using namespace sm100;
  const bool rope = p.theta > 0.f;
  const float scale = rsqrtf((float)p.dh);
  for (int kv = j; kv < p.Hkv; kv += cps) {
    uint8_t *img = p.qimg + ((size_t)b * p.Hkv + kv) * kQueryOperandBytes;
    // rows that carry no query stay zero: G..7 and 8+G..15, 16 pieces of 16 bytes each
    for (int i = t; i < 2 * (8 - p.Gq) * 16; i += n_threads) {
      const int row = (i >> 4) < 8 - p.Gq ? p.Gq + (i >> 4) : 8 + p.Gq + ((i >> 4) - (8 - p.Gq));
      const int piece = i & 15;
      *reinterpret_cast<uint4 *>(img + (size_t)(piece >> 3) * 2048 + (row >> 3) * 1024 + (row & 7) * 128 + (piece & 7) * 16) =
          make_uint4(0, 0, 0, 0);
    }
    for (int i = t; i < p.Gq * p.dh; i += n_threads) {
      const int g = i >> 7, c = i & 127;  // d_h = 128 on this path
      const __nv_bfloat16 *qp = p.q + ((size_t)b * p.Hq + (size_t)kv * p.Gq + g) * p.dh;
      float v = __bfloat162float(qp[c]);
      if (rope) {
        const float o = __bfloat162float(qp[c ^ 64]);
        float sn, cs;
        rope_sincos(p.sinks + L - 1, p.rope_turns[c & 63], sn, cs);
        v = c < 64 ? v * cs - o * sn : v * cs + o * sn;
      }
      v *= scale;
      const __nv_bfloat16 hi = __float2bfloat16_rn(v);
      const __nv_bfloat16 lo = __float2bfloat16_rn(v - __bfloat162float(hi));
      *reinterpret_cast<__nv_bfloat16 *>(img + query_operand_offset(g, c)) = hi;
      *reinterpret_cast<__nv_bfloat16 *>(img + query_operand_offset(8 + g, c)) = lo;
    }
  }
}

}  // namespace s4r
