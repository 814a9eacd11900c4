// Causal grouped-query attention of the prefill path (flash-style, one pass over the keys).
//
// One CTA per (64-query tile, query head, sequence); 4 warps of 16 query rows.  K/V tiles of 64
// keys are staged in shared memory with cp.async straight from the KV cache the QKV epilogue
// just filled; S = Q K^T and O += P V run on mma.sync m16n8k16 with fp32 online softmax in
// registers.  Query p attends keys t <= p; query head h uses kv head h / (Hq / Hkv).  The cache holds binary16
// keys and values, so the query (hi + lo pair) and the probabilities enter the MMAs as binary16 too; the output
// leaves as a bf16 hi + lo pair, the operand type of the output projection.
#include "common.cuh"
#include "kernels.h"

namespace ladder {
namespace {

constexpr int kQT = 64, kKT = 64, kPfThreads = 128;

__device__ __forceinline__ void cp16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}

// SPLIT: the query comes as a binary16 hi + lo pair and the output is written as a bf16 one (value ~ hi + lo).
template <int DH, bool SPLIT>
__global__ void __launch_bounds__(kPfThreads) prefill_attention_kernel(const __half* __restrict__ q,
                                                                       const __half* __restrict__ q_lo,
                                                                       const kv_t* __restrict__ kc,
                                                                       const kv_t* __restrict__ vc, int seq_len,
                                                                       int n_q_heads, int n_kv_heads, int max_seq_len,
                                                                       __nv_bfloat16* __restrict__ o,
                                                                       __nv_bfloat16* __restrict__ o_lo, const int pos0,
                                                                       const int out_f16,
                                                                       const int32_t* __restrict__ lens) {
  constexpr int P = DH + 8;  // smem pitch in elements
  extern __shared__ __align__(128) uint8_t smem_raw[];
  __half* sQ = reinterpret_cast<__half*>(smem_raw);
  __half* sK = sQ + kQT * P;
  __half* sV = sK + kKT * P;
  __half* sQl = sV + kKT * P;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tig = lane & 3;
  const int q0 = blockIdx.x * kQT, h = blockIdx.y, b = blockIdx.z;
  const int kvh = h / (n_q_heads / n_kv_heads);
  const size_t qrow_stride = static_cast<size_t>(n_q_heads) * DH;
  const kv_t* kg = kc + (static_cast<size_t>(b) * n_kv_heads + kvh) * max_seq_len * DH;
  const kv_t* vg = vc + (static_cast<size_t>(b) * n_kv_heads + kvh) * max_seq_len * DH;
  constexpr int CPR = DH / 8;  // 16-byte chunks per row
  const int len_b = lens ? min(max(lens[b], 0), seq_len) : seq_len;  // valid rows of this sequence
  if (q0 >= len_b) return;                                           // a tile of padding rows

  for (int i = tid; i < kQT * CPR; i += kPfThreads) {
    const int r = i / CPR, c = i % CPR;
    const bool v = q0 + r < len_b;
    const size_t off = (static_cast<size_t>(b) * seq_len) * qrow_stride + static_cast<size_t>(h) * DH +
                       (v ? static_cast<size_t>(q0 + r) * qrow_stride + c * 8 : 0);
    cp16(smem_u32(sQ + r * P + c * 8), q + off, v);
    if (SPLIT) cp16(smem_u32(sQl + r * P + c * 8), q_lo + off, v);
  }
  asm volatile("cp.async.commit_group;" ::: "memory");

  float oacc[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i)
#pragma unroll
    for (int c = 0; c < 4; ++c) oacc[i][c] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  const float scale = rsqrtf(static_cast<float>(DH));
  const int q_hi = min(q0 + kQT, len_b) - 1;    // last valid query of the tile
  const int n_keys = pos0 + len_b;              // cache rows that exist for this call
  const int n_kt = (pos0 + q_hi) / kKT + 1;

  for (int kt = 0; kt < n_kt; ++kt) {
    __syncthreads();  // previous tile fully consumed
    for (int i = tid; i < kKT * CPR; i += kPfThreads) {
      const int r = i / CPR, c = i % CPR;
      const int key = kt * kKT + r;
      const bool v = key < n_keys;
      const size_t off = v ? static_cast<size_t>(key) * DH + c * 8 : 0;
      cp16(smem_u32(sK + r * P + c * 8), kg + off, v);
      cp16(smem_u32(sV + r * P + c * 8), vg + off, v);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();

    // S = Q K^T  (16 x 64 per warp)
    float s[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int c = 0; c < 4; ++c) s[i][c] = 0.f;
#pragma unroll
    for (int ks = 0; ks < DH; ks += 16) {
      uint32_t a0, a1, a2, a3, l0 = 0, l1 = 0, l2 = 0, l3 = 0;
      ldsm_x4(smem_u32(sQ + (warp * 16 + (lane & 15)) * P + ks + (lane >> 4) * 8), a0, a1, a2, a3);
      if (SPLIT) ldsm_x4(smem_u32(sQl + (warp * 16 + (lane & 15)) * P + ks + (lane >> 4) * 8), l0, l1, l2, l3);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4(smem_u32(sK + (j * 16 + (lane & 7) + (lane >> 4) * 8) * P + ks + ((lane >> 3) & 1) * 8), b0, b1, b2, b3);
        mma_f16_16816(s[2 * j], a0, a1, a2, a3, b0, b1);
        mma_f16_16816(s[2 * j + 1], a0, a1, a2, a3, b2, b3);
        if (SPLIT) {
          mma_f16_16816(s[2 * j], l0, l1, l2, l3, b0, b1);
          mma_f16_16816(s[2 * j + 1], l0, l1, l2, l3, b2, b3);
        }
      }
    }

    // scale, causal mask, online softmax (rows g and g+8 of the warp's 16)
    const int qa = q0 + warp * 16 + g;
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int key = kt * kKT + i * 8 + tig * 2 + (c & 1);
        const int qi = pos0 + qa + (c >> 1) * 8;  // the query's position
        const float v = (key <= qi && key < n_keys) ? s[i][c] * scale : -INFINITY;
        s[i][c] = v;
        mx[c >> 1] = fmaxf(mx[c >> 1], v);
      }
    float corr[2], mnew[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      mnew[r] = fmaxf(m_run[r], mx[r]);
      corr[r] = (m_run[r] == -INFINITY) ? 0.f : __expf(m_run[r] - mnew[r]);
      m_run[r] = mnew[r];
    }
    float rs[2] = {0.f, 0.f};
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const float mref = mnew[c >> 1];
        const float e = (mref == -INFINITY) ? 0.f : __expf(s[i][c] - mref);
        s[i][c] = e;
        rs[c >> 1] += e;
      }
#pragma unroll
    for (int r = 0; r < 2; ++r) l_run[r] = l_run[r] * corr[r] + rs[r];
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
      oacc[i][0] *= corr[0];
      oacc[i][1] *= corr[0];
      oacc[i][2] *= corr[1];
      oacc[i][3] *= corr[1];
    }

    // O += P V
#pragma unroll
    for (int kk = 0; kk < kKT / 16; ++kk) {
      const uint32_t a0 = pack_f16x2(s[2 * kk][0], s[2 * kk][1]);
      const uint32_t a1 = pack_f16x2(s[2 * kk][2], s[2 * kk][3]);
      const uint32_t a2 = pack_f16x2(s[2 * kk + 1][0], s[2 * kk + 1][1]);
      const uint32_t a3 = pack_f16x2(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
      for (int d = 0; d < DH / 16; ++d) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(smem_u32(sV + (kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * P + d * 16 + (lane >> 4) * 8), b0, b1,
                  b2, b3);
        mma_f16_16816(oacc[2 * d], a0, a1, a2, a3, b0, b1);
        mma_f16_16816(oacc[2 * d + 1], a0, a1, a2, a3, b2, b3);
      }
    }
  }

  // finalise: divide by the row sums (reduced over the quad) and store bf16
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int qi = q0 + warp * 16 + g + r * 8;
    if (qi >= len_b) continue;
    const float inv = l_run[r] > 0.f ? 1.f / l_run[r] : 0.f;
    const size_t doff = (static_cast<size_t>(b) * seq_len + qi) * qrow_stride + static_cast<size_t>(h) * DH;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
      const float v0 = oacc[i][2 * r] * inv, v1 = oacc[i][2 * r + 1] * inv;
      if (out_f16) {  // one binary16 value per element: the operand of the binary16 output projection
        *reinterpret_cast<uint32_t*>(o + doff + i * 8 + tig * 2) = pack_f16x2(v0, v1);
        continue;
      }
      const uint32_t hi = pack_bf16x2(v0, v1);
      *reinterpret_cast<uint32_t*>(o + doff + i * 8 + tig * 2) = hi;
      if (SPLIT) *reinterpret_cast<uint32_t*>(o_lo + doff + i * 8 + tig * 2) = pack_bf16x2(v0 - bf16_lo(hi), v1 - bf16_hi(hi));
    }
  }
}

template <int DH, bool SPLIT>
cudaError_t launch_dh(const __half* q, const __half* q_lo, const kv_t* k, const kv_t* v,
                      int batch, int seq_len, int n_q_heads, int n_kv_heads, int max_seq_len, __nv_bfloat16* o,
                      __nv_bfloat16* o_lo, cudaStream_t stream, int pos0, int out_f16, const int32_t* lens) {
  constexpr int smem = 4 * 64 * (DH + 8) * 2;
  dim3 grid((seq_len + kQT - 1) / kQT, n_q_heads, batch);
  prefill_attention_kernel<DH, SPLIT><<<grid, kPfThreads, smem, stream>>>(q, q_lo, k, v, seq_len, n_q_heads, n_kv_heads,
                                                                          max_seq_len, o, o_lo, pos0, out_f16, lens);
  return cudaGetLastError();
}

template <int DH, bool SPLIT>
cudaError_t init_dh() {
  return cudaFuncSetAttribute(prefill_attention_kernel<DH, SPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              4 * 64 * (DH + 8) * 2);
}

}  // namespace

cudaError_t prefill_attention_init() {
  cudaError_t e = init_dh<128, true>();
  if (e == cudaSuccess) e = init_dh<128, false>();
  if (e == cudaSuccess) e = init_dh<64, true>();
  if (e == cudaSuccess) e = init_dh<64, false>();
  return e;
}

cudaError_t launch_prefill_attention(const __half* q, const __half* q_lo, const kv_t* k,
                                     const kv_t* v, int batch, int seq_len, int n_q_heads, int n_kv_heads,
                                     int head_dim, int max_seq_len, __nv_bfloat16* o, __nv_bfloat16* o_lo,
                                     cudaStream_t stream, int pos0, bool out_f16, const int32_t* lens) {
  const bool split = q_lo != nullptr && (o_lo != nullptr || out_f16);
  if (out_f16 && o_lo) return cudaErrorInvalidValue;
  const int of = out_f16 ? 1 : 0;
  if (pos0 < 0 || pos0 + seq_len > max_seq_len) return cudaErrorInvalidValue;
  if (head_dim == 128)
    return split ? launch_dh<128, true>(q, q_lo, k, v, batch, seq_len, n_q_heads, n_kv_heads, max_seq_len, o, o_lo, stream, pos0, of, lens)
                 : launch_dh<128, false>(q, q_lo, k, v, batch, seq_len, n_q_heads, n_kv_heads, max_seq_len, o, o_lo, stream, pos0, of, lens);
  if (head_dim == 64)
    return split ? launch_dh<64, true>(q, q_lo, k, v, batch, seq_len, n_q_heads, n_kv_heads, max_seq_len, o, o_lo, stream, pos0, of, lens)
                 : launch_dh<64, false>(q, q_lo, k, v, batch, seq_len, n_q_heads, n_kv_heads, max_seq_len, o, o_lo, stream, pos0, of, lens);
  return cudaErrorInvalidValue;
}

}  // namespace ladder
