// Grouped-query decode attention, split over the KV cache.
//
// One CTA per (split s, group of GT query heads sharing a kv head, sequence b).  The CTA
//   1. computes the GT x CH score block with mma.sync (Q padded to 16 rows is the A operand,
//      K rows are read straight from the cache as B fragments -- the contraction index is
//      permuted identically on both sides so each thread reads 16 contiguous bytes of a key),
//   2. does the softmax of its block in fp32 (max, exp, sum) in shared memory,
//   3. accumulates P.V on the CUDA cores (each warp walks keys, each lane owns Dh/32 dims),
//   4. writes (o, m, l) partials to an L2-resident scratch, and the LAST CTA of a head group to
//      arrive (atomic ticket, no spinning) merges the partials by log-sum-exp in a fixed order
//      and writes o in fp32.  The ticket counters clean themselves up for the next launch.
// The kernel is latency- not bandwidth-bound (KV is ~1 % of the bytes of a decode step); its
// shared-memory footprint is kept small so it can co-reside with a weight-streaming GEMM CTA.
#include "common.cuh"
#include "kernels.h"

namespace ladder {
namespace {

constexpr int kAttnThreads = 128;
constexpr int kMaxChunk = 256;

template <int GT, int DH>
__global__ void __launch_bounds__(kAttnThreads) decode_attention_kernel(const DecodeAttnParams p, int chunk,
                                                                        int32_t* counters) {
  constexpr int DPL = DH / 32;  // dims per lane in the P.V phase
  constexpr int KJ = DH / 32;   // 16-byte loads per key per thread in the score phase
  __shared__ float sc[GT][kMaxChunk];
  __shared__ float red[4][GT][DH];
  __shared__ float ml[GT][2];
  __shared__ int last_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, tig = lane & 3;
  const int split = blockIdx.x, hg = blockIdx.y, b = blockIdx.z;
  const int head0 = hg * GT;
  const int group = p.n_q_heads / p.n_kv_heads;
  const int kvh = head0 / group;
  const size_t kv_base = (static_cast<size_t>(b) * p.n_kv_heads + kvh) * p.max_seq_len * DH;
  const __nv_bfloat16* K = p.k + kv_base;
  const __nv_bfloat16* V = p.v + kv_base;

  pdl_launch_dependents();
  pdl_wait();

  int L = p.kv_len[b] + p.kv_len_offset;
  L = max(0, min(L, p.max_seq_len));
  const int k_begin = min(split * chunk, L);
  const int k_end = min(k_begin + chunk, L);
  const int nk = k_end - k_begin;
  const float scale = rsqrtf(static_cast<float>(DH));

  // ---- 1. scores
  // q as a bf16 hi + lo pair (q ~ hi + lo), so the fp32 query loses nothing on its way into the MMA
  uint32_t qa[KJ][2][2], ql[KJ][2][2];  // [j][half][pair]: q[head0+g][j*32 + tig*8 + half*4 + 2*pair ..+1]
#pragma unroll
  for (int j = 0; j < KJ; ++j)
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float4 v = make_float4(0, 0, 0, 0);
      if (g < GT)
        v = *reinterpret_cast<const float4*>(p.q + (static_cast<size_t>(b) * p.n_q_heads + head0 + g) * DH + j * 32 +
                                             tig * 8 + h * 4);
      qa[j][h][0] = pack_bf16x2(v.x, v.y);
      qa[j][h][1] = pack_bf16x2(v.z, v.w);
      ql[j][h][0] = pack_bf16x2(v.x - bf16_lo(qa[j][h][0]), v.y - bf16_hi(qa[j][h][0]));
      ql[j][h][1] = pack_bf16x2(v.z - bf16_lo(qa[j][h][1]), v.w - bf16_hi(qa[j][h][1]));
    }
  for (int kb = warp * 8; kb < nk; kb += 32) {
    const int key = k_begin + kb + g;
    float c[4] = {0.f, 0.f, 0.f, 0.f};
    uint4 kf[KJ];
#pragma unroll
    for (int j = 0; j < KJ; ++j)
      kf[j] = (kb + g < nk) ? *reinterpret_cast<const uint4*>(K + static_cast<size_t>(key) * DH + j * 32 + tig * 8)
                            : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int j = 0; j < KJ; ++j) {
      mma_bf16_16816(c, qa[j][0][0], 0u, qa[j][0][1], 0u, kf[j].x, kf[j].y);
      mma_bf16_16816(c, qa[j][1][0], 0u, qa[j][1][1], 0u, kf[j].z, kf[j].w);
      mma_bf16_16816(c, ql[j][0][0], 0u, ql[j][0][1], 0u, kf[j].x, kf[j].y);
      mma_bf16_16816(c, ql[j][1][0], 0u, ql[j][1][1], 0u, kf[j].z, kf[j].w);
    }
    if (g < GT) {
      const int c0 = kb + 2 * tig;
      if (c0 < nk) sc[g][c0] = c[0] * scale;
      if (c0 + 1 < nk) sc[g][c0 + 1] = c[1] * scale;
    }
  }
  __syncthreads();

  // ---- 2. softmax of the block (fp32)
  for (int h = warp; h < GT; h += 4) {
    float m = -INFINITY;
    for (int i = lane; i < nk; i += 32) m = fmaxf(m, sc[h][i]);
    m = warp_max(m);
    float l = 0.f;
    for (int i = lane; i < nk; i += 32) {
      const float e = __expf(sc[h][i] - m);
      sc[h][i] = e;
      l += e;
    }
    l = warp_sum(l);
    if (lane == 0) {
      ml[h][0] = m;
      ml[h][1] = l;
    }
  }
  __syncthreads();

  // ---- 3. P.V
  float acc[GT][DPL];
#pragma unroll
  for (int h = 0; h < GT; ++h)
#pragma unroll
    for (int d = 0; d < DPL; ++d) acc[h][d] = 0.f;
  for (int i = warp; i < nk; i += 4) {
    const __nv_bfloat16* vr = V + static_cast<size_t>(k_begin + i) * DH + lane * DPL;
    float v[DPL];
    if (DPL == 4) {
      const uint2 u = *reinterpret_cast<const uint2*>(vr);
      v[0] = bf16_lo(u.x);
      v[1] = bf16_hi(u.x);
      v[DPL - 2] = bf16_lo(u.y);
      v[DPL - 1] = bf16_hi(u.y);
    } else {
      const uint32_t u = *reinterpret_cast<const uint32_t*>(vr);
      v[0] = bf16_lo(u);
      v[1] = bf16_hi(u);
    }
#pragma unroll
    for (int h = 0; h < GT; ++h) {
      const float pw = sc[h][i];
#pragma unroll
      for (int d = 0; d < DPL; ++d) acc[h][d] += pw * v[d];
    }
  }
#pragma unroll
  for (int h = 0; h < GT; ++h)
#pragma unroll
    for (int d = 0; d < DPL; ++d) red[warp][h][lane * DPL + d] = acc[h][d];
  __syncthreads();

  // ---- 4. partial -> scratch
  const int stride = DH + 2;
  for (int idx = tid; idx < GT * DH; idx += kAttnThreads) {
    const int h = idx / DH, d = idx % DH;
    const float o = red[0][h][d] + red[1][h][d] + red[2][h][d] + red[3][h][d];
    p.scratch[((static_cast<size_t>(b) * p.n_q_heads + head0 + h) * p.n_splits + split) * stride + d] = o;
  }
  if (tid < GT) {
    float* dst = p.scratch + ((static_cast<size_t>(b) * p.n_q_heads + head0 + tid) * p.n_splits + split) * stride + DH;
    dst[0] = ml[tid][0];
    dst[1] = ml[tid][1];
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    int32_t* ctr = counters + b * gridDim.y + hg;
    const int ticket = atomicAdd(ctr, 1);
    last_s = (ticket == p.n_splits - 1);
    if (last_s) *ctr = 0;  // every CTA of this group has arrived: reset for the next launch
  }
  __syncthreads();
  if (!last_s) return;
  __threadfence();

  // ---- 5. merge (fixed order over splits => deterministic)
  for (int idx = tid; idx < GT * DH; idx += kAttnThreads) {
    const int h = idx / DH, d = idx % DH;
    const float* base = p.scratch + (static_cast<size_t>(b) * p.n_q_heads + head0 + h) * p.n_splits * stride;
    float M = -INFINITY;
    for (int s = 0; s < p.n_splits; ++s) M = fmaxf(M, __ldcg(base + s * stride + DH));
    float lsum = 0.f, o = 0.f;
    for (int s = 0; s < p.n_splits; ++s) {
      const float ms = __ldcg(base + s * stride + DH);
      const float w = (ms == -INFINITY) ? 0.f : __expf(ms - M);
      lsum += w * __ldcg(base + s * stride + DH + 1);
      o += w * __ldcg(base + s * stride + d);
    }
    p.o[(static_cast<size_t>(b) * p.n_q_heads + head0 + h) * DH + d] = lsum > 0.f ? o / lsum : 0.f;
  }
}

template <int GT>
cudaError_t launch_gt(const DecodeAttnParams& p, int chunk, int32_t* counters, cudaStream_t stream, bool pdl) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.n_splits, p.n_q_heads / GT, p.batch);
  cfg.blockDim = dim3(kAttnThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  if (p.head_dim == 128) return cudaLaunchKernelEx(&cfg, decode_attention_kernel<GT, 128>, p, chunk, counters);
  return cudaLaunchKernelEx(&cfg, decode_attention_kernel<GT, 64>, p, chunk, counters);
}

int heads_per_cta(int n_q_heads, int n_kv_heads) {
  const int group = n_q_heads / n_kv_heads;
  int gt = 1;
  while (gt < 8 && group % (gt * 2) == 0) gt *= 2;
  return gt;
}

}  // namespace

int decode_attention_splits(int batch, int n_kv_heads, int max_len, int sm_count) {
  // enough CTAs for ~2 per SM, at most kMaxChunk keys per CTA, at least 32
  const int ctas_per_split = batch * n_kv_heads;
  int want = (2 * sm_count + ctas_per_split - 1) / ctas_per_split;
  const int lo = (max_len + kMaxChunk - 1) / kMaxChunk;
  const int hi = (max_len + 31) / 32;
  if (want < lo) want = lo;
  if (want > hi) want = hi;
  return want < 1 ? 1 : want;
}

// scratch layout: [batch * Hq ticket counters (int32), padded to 64 floats][partials]
size_t decode_attention_scratch_floats(int batch, int n_q_heads, int head_dim, int n_splits) {
  const size_t counters = (static_cast<size_t>(batch) * n_q_heads + 63) / 64 * 64;
  return counters + static_cast<size_t>(batch) * n_q_heads * n_splits * (head_dim + 2);
}

cudaError_t launch_decode_attention(const DecodeAttnParams& p_in, cudaStream_t stream, bool pdl) {
  DecodeAttnParams p = p_in;
  const size_t counters = (static_cast<size_t>(p.batch) * p.n_q_heads + 63) / 64 * 64;
  int32_t* ctr = reinterpret_cast<int32_t*>(p.scratch);
  p.scratch = p.scratch + counters;
  int chunk = (p.max_len + p.n_splits - 1) / p.n_splits;
  chunk = (chunk + 31) / 32 * 32;
  if (chunk > kMaxChunk) return cudaErrorInvalidValue;
  switch (heads_per_cta(p.n_q_heads, p.n_kv_heads)) {
    case 8: return launch_gt<8>(p, chunk, ctr, stream, pdl);
    case 4: return launch_gt<4>(p, chunk, ctr, stream, pdl);
    case 2: return launch_gt<2>(p, chunk, ctr, stream, pdl);
    default: return launch_gt<1>(p, chunk, ctr, stream, pdl);
  }
}

}  // namespace ladder
