// Epilogue of the prefill GEMMs: the accumulator pair (m, n), (m, n+1) -- n even -- goes through the fused tail of
// its layer step.
#pragma once
#include "common.cuh"
#include "kernels.h"

namespace ladder {

__device__ __forceinline__ void epilogue_pair(const LargeMParams& p, int m, int n, float v0, float v1) {
  if (m >= p.M || n >= p.N) return;
  switch (p.epi_mode) {
    case EPI_RESID: {
      const size_t o = static_cast<size_t>(m) * p.N + n;
      const float2 a = *reinterpret_cast<const float2*>(p.addend + o);
      *reinterpret_cast<float2*>(static_cast<float*>(p.out) + o) = make_float2(a.x + v0, a.y + v1);
      break;
    }
    case EPI_SWIGLU: {
      const float h = v0 / (1.f + __expf(-v0)) * v1;
      const size_t o = static_cast<size_t>(m) * (p.N >> 1) + (n >> 1);
      if (p.f16) {  // one binary16 value, saturating
        static_cast<__half*>(p.out)[o] = __float2half_rn(fminf(fmaxf(h, -65504.f), 65504.f));
        break;
      }
      const __nv_bfloat16 hi = __float2bfloat16_rn(h);
      static_cast<__nv_bfloat16*>(p.out)[o] = hi;
      if (p.out_lo) p.out_lo[o] = __float2bfloat16_rn(h - __bfloat162float(hi));
      break;
    }
    case EPI_PLAIN:
      *reinterpret_cast<float2*>(static_cast<float*>(p.out) + static_cast<size_t>(m) * p.N + n) = make_float2(v0, v1);
      break;
    case EPI_BF16: {
      const size_t o = static_cast<size_t>(m) * p.N + n;
      if (p.f16) {
        *reinterpret_cast<uint32_t*>(static_cast<__half*>(p.out) + o) = pack_kv(v0, v1);
        break;
      }
      const uint32_t hi = pack_bf16x2(v0, v1);
      *reinterpret_cast<uint32_t*>(static_cast<__nv_bfloat16*>(p.out) + o) = hi;
      if (p.out_lo) *reinterpret_cast<uint32_t*>(p.out_lo + o) = pack_bf16x2(v0 - bf16_lo(hi), v1 - bf16_hi(hi));
      break;
    }
    case EPI_QKV_ROPE: {
      const QkvEpilogue& e = p.qkv;
      const int Dh = e.head_dim, nq = e.n_q_heads * Dh, nk = e.n_kv_heads * Dh;
      const int b = m / e.prefill_seq_len, pos = e.prefill_pos0 + m % e.prefill_seq_len;
      if (n < nq + nk) {
        const float2 cs = e.rope[static_cast<size_t>(pos) * (Dh >> 1) + ((n % Dh) >> 1)];
        const float a0 = v0 * cs.x - v1 * cs.y, a1 = v0 * cs.y + v1 * cs.x;
        v0 = a0;
        v1 = a1;
      }
      if (n < nq) {
        const uint32_t hi = pack_f16x2(v0, v1);      // the query as the attention's binary16 operand pair
        *reinterpret_cast<uint32_t*>(e.q_out_f16 + static_cast<size_t>(m) * nq + n) = hi;
        if (e.q_out_lo)
          *reinterpret_cast<uint32_t*>(e.q_out_lo + static_cast<size_t>(m) * nq + n) =
              pack_f16x2(v0 - f16_lo(hi), v1 - f16_hi(hi));
      } else {
        if (e.prefill_lens && m % e.prefill_seq_len >= e.prefill_lens[b]) break;  // padding row: nothing to cache
        const int nn = n < nq + nk ? n - nq : n - nq - nk;
        kv_t* cache = n < nq + nk ? e.k_cache : e.v_cache;
        const size_t off = ((static_cast<size_t>(b) * e.n_kv_heads + nn / Dh) * e.max_seq_len + pos) * Dh + (nn % Dh);
        *reinterpret_cast<uint32_t*>(cache + off) = pack_kv(v0, v1);
      }
      break;
    }
    default: break;
  }
}

}  // namespace ladder
