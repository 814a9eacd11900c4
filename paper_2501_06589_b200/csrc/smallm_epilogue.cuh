// Epilogues shared by the weight-streaming decode GEMM kernels.  `value(r, b)` returns the finished
// accumulator (K-split reduced, 1/rms applied) of local row r of the block and batch row b; NT
// threads (index ct) walk the block's outputs.
#pragma once
#include "common.cuh"
#include "kernels.h"

namespace ladder {

// Second copy of an output value as the next GEMM's MMA operand: bf16 high part in row b, low part in row 4 + b
// of the 2048-wide chunk that column n falls in (the layout the persistent kernel's activation buffer has).
__device__ __forceinline__ void store_packed(__nv_bfloat16* pack, const __nv_bfloat16* gain, int b, int n, float v) {
  if (gain) v *= __bfloat162float(gain[n]);
  const __nv_bfloat16 hi = __float2bfloat16_rn(v);
  const __nv_bfloat16 lo = __float2bfloat16_rn(v - __bfloat162float(hi));
  __nv_bfloat16* dst = pack + (static_cast<size_t>(n >> 11) * 8 + b) * 2048 + (n & 2047);
  dst[0] = hi;
  dst[4 * 2048] = lo;
}

template <int NT = 128, typename ValueFn>
__device__ __forceinline__ void smallm_epilogue(const SmallMParams& p, int ct, int prow, int nbase, int batch,
                                                ValueFn value) {
  if (p.epi_mode == EPI_RESID || p.epi_mode == EPI_PLAIN) {
    // x_m = addend + h_m(.)   (the residual add of Eq. 1 / Eq. 2 of the paper), or a plain store
    float* out = static_cast<float*>(p.out);
    for (int idx = ct; idx < prow * batch; idx += NT) {
      const int r = idx % prow, b = idx / prow;
      const size_t o = static_cast<size_t>(b) * p.N + nbase + r;
      float v = value(r, b);
      if (p.epi_mode == EPI_RESID) v += __ldcg(p.addend + o);  // L2: may have been written by another SM of this launch
      out[o] = v;
      if (p.pack_out) store_packed(p.pack_out, p.pack_gain, b, nbase + r, v);
    }
  } else if (p.epi_mode == EPI_SWIGLU) {
    // rows (2j, 2j+1) = (gate_j, up_j)  ->  h_j = silu(gate_j) * up_j
    float* out = static_cast<float*>(p.out);
    const int half = prow >> 1;
    for (int idx = ct; idx < half * batch; idx += NT) {
      const int pr = idx % half, b = idx / half;
      const float gt = value(2 * pr, b), up = value(2 * pr + 1, b);
      const float hv = gt / (1.f + __expf(-gt)) * up;
      out[static_cast<size_t>(b) * (p.N >> 1) + ((nbase >> 1) + pr)] = hv;
      if (p.pack_out) store_packed(p.pack_out, p.pack_gain, b, (nbase >> 1) + pr, hv);
    }
  } else if (p.epi_mode == EPI_QKV_ROPE) {
    // rotary embedding on interleaved pairs of q and k at position seq_lens[b]; k, v appended to the cache
    const QkvEpilogue& e = p.qkv;
    const int half = prow >> 1, Dh = e.head_dim;
    const int nq = e.n_q_heads * Dh, nk = e.n_kv_heads * Dh;
    for (int idx = ct; idx < half * batch; idx += NT) {
      const int pr = idx % half, b = idx / half;
      const int n = nbase + 2 * pr;
      float v0 = value(2 * pr, b), v1 = value(2 * pr + 1, b);
      const int pos = e.seq_lens[b];
      if (pos < 0 || pos >= e.max_seq_len) {
        if (p.status) atomicOr(p.status, LADDER_DEV_CACHE_OVERFLOW);
        continue;
      }
      if (n < nq + nk) {
        const float2 cs = e.rope[static_cast<size_t>(pos) * (Dh >> 1) + ((n % Dh) >> 1)];
        const float a0 = v0 * cs.x - v1 * cs.y, a1 = v0 * cs.y + v1 * cs.x;
        v0 = a0;
        v1 = a1;
      }
      if (n < nq) {
        *reinterpret_cast<float2*>(e.q_out_f32 + static_cast<size_t>(b) * nq + n) = make_float2(v0, v1);
      } else {
        const int nn = n < nq + nk ? n - nq : n - nq - nk;
        kv_t* cache = n < nq + nk ? e.k_cache : e.v_cache;
        const size_t off = ((static_cast<size_t>(b) * e.n_kv_heads + nn / Dh) * e.max_seq_len + pos) * Dh + (nn % Dh);
        *reinterpret_cast<uint32_t*>(cache + off) = pack_kv(v0, v1);
      }
    }
  }
}

}  // namespace ladder
