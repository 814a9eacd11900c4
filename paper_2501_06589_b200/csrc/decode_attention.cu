// Grouped-query decode attention, split over the KV cache.
//
// The step is latency-bound, not bandwidth-bound (the KV prefix is ~1 % of the bytes of a decode
// step), so the kernel is built around memory-level parallelism: one CTA per (64-key split, group
// of GT query heads sharing a kv head, sequence); each of its 4 warps owns 16 keys and issues ALL of
// its loads -- q, 16 key rows as MMA fragments, 16 value rows -- before the first dependent
// instruction, so the whole CTA costs about one memory round trip plus one merge.
//   1. scores: mma.sync with Q (padded to 16 rows, binary16 hi + lo pair so the fp32 query loses
//      nothing) as the A operand and key rows read straight from the cache as B fragments (the
//      contraction index is permuted identically on both sides: 16 contiguous bytes per thread);
//   2. fp32 softmax statistics per warp, probabilities to shared memory;
//   3. P.V on the CUDA cores in fp32 from the value rows already in registers (batch <= 8), or on mma.sync
//      with the probabilities as a binary16 hi + lo pair (batch > 8: see PVMMA below);
//   4. the 4 warps are merged by log-sum-exp in shared memory and the CTA's (o, m, l) partial goes
//      to an L2-resident scratch; a second, tiny kernel (one CTA per sequence and head, launched
//      with programmatic dependent launch) merges the splits in a fixed order and writes o in fp32.
// The shared-memory footprint (~19 KB) lets a CTA co-reside with a weight-streaming GEMM CTA.
#include "../../include/ladder.h"
#include "common.cuh"
#include "kernels.h"

namespace ladder {
namespace {

constexpr int kAttnThreads = 128;
constexpr int kChunk = 64;  // keys per CTA (16 per warp)

// PVMMA (used for batch > 8, where the step stops being latency-bound and this kernel became issue-bound on its
// CUDA-core P.V loop: 65 % issue-slot use at 2.7 TB/s): P.V runs on mma.sync too.  The probabilities of head g
// are already laid out as the A fragment (the score MMA's C fragment, as a binary16 hi + lo pair), and a lane reads
// the value rows as 32-bit words V[key][16 j + 2 g, +1] for its four keys 2t, 2t+1, 2t+8, 2t+9, so that two byte
// permutes turn them into the B fragments of an "even dims" and an "odd dims" MMA per 16 dims.
template <int GT, int DH, bool PVMMA>
__global__ void __launch_bounds__(kAttnThreads) decode_attention_kernel(const DecodeAttnParams p) {
  constexpr int DPL = DH / 32;  // dims per lane in the P.V phase
  constexpr int KJ = DH / 32;   // 16-byte loads per key per thread in the score phase
  __shared__ __align__(16) float ps[4][GT][16];
  __shared__ float red[4][GT][DH];
  __shared__ float mls[4][GT][2];
  __shared__ float mfac[GT][4];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, tig = lane & 3;
  const int split = blockIdx.x, hg = blockIdx.y, b = blockIdx.z;
  const int head0 = hg * GT;
  const int group = p.n_q_heads / p.n_kv_heads;
  const int kvh = head0 / group;
  const size_t kv_base = (static_cast<size_t>(b) * p.n_kv_heads + kvh) * p.max_seq_len * DH;
  const kv_t* K = p.k + kv_base;
  const kv_t* V = p.v + kv_base;

  pdl_launch_dependents();
  pdl_wait();

  int L = p.kv_len[b] + p.kv_len_offset;
  L = max(0, min(L, p.max_seq_len));
  const int kw0 = split * kChunk + warp * 16;  // first key of this warp
  const float scale = rsqrtf(static_cast<float>(DH));

  // ---- all loads up front
  uint4 kf[2][KJ];
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
    const int key = kw0 + nt * 8 + g;
#pragma unroll
    for (int j = 0; j < KJ; ++j)
      kf[nt][j] = key < L ? *reinterpret_cast<const uint4*>(K + static_cast<size_t>(key) * DH + j * 32 + tig * 8)
                          : make_uint4(0, 0, 0, 0);
  }
  uint32_t vr[16][DPL / 2];
  if constexpr (PVMMA) {  // [j][q] = V[kw0 + key(q)][16 j + 2 g, +1], key(q) = 2 tig + (q & 1) + 8 (q >> 1)
#pragma unroll
    for (int q4 = 0; q4 < 4; ++q4) {
      const int key = kw0 + 2 * tig + (q4 & 1) + 8 * (q4 >> 1);
#pragma unroll
      for (int j = 0; j < DH / 16; ++j) {
        const int i = j * 4 + q4;
        vr[i / (DPL / 2)][i % (DPL / 2)] =
            key < L ? *reinterpret_cast<const uint32_t*>(V + static_cast<size_t>(key) * DH + 16 * j + 2 * g) : 0u;
      }
    }
  }
#pragma unroll
  for (int i = 0; i < (PVMMA ? 0 : 16); ++i) {
    const int key = kw0 + i;
    if (DPL == 4) {
      const uint2 u = key < L ? *reinterpret_cast<const uint2*>(V + static_cast<size_t>(key) * DH + lane * DPL)
                              : make_uint2(0, 0);
      vr[i][0] = u.x;
      vr[i][DPL / 2 - 1] = u.y;
    } else {
      vr[i][0] = key < L ? *reinterpret_cast<const uint32_t*>(V + static_cast<size_t>(key) * DH + lane * DPL) : 0u;
    }
  }
  // q as a binary16 hi + lo pair (the keys' type): [j][half][pair] covers q[head0+g][j*32 + tig*8 + half*4 + 2*pair ..+1]
  uint32_t qa[KJ][2][2], ql[KJ][2][2];
#pragma unroll
  for (int j = 0; j < KJ; ++j)
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float4 v = make_float4(0, 0, 0, 0);
      if (g < GT)
        v = *reinterpret_cast<const float4*>(p.q + (static_cast<size_t>(b) * p.n_q_heads + head0 + g) * DH + j * 32 +
                                             tig * 8 + h * 4);
      qa[j][h][0] = pack_f16x2(v.x, v.y);
      qa[j][h][1] = pack_f16x2(v.z, v.w);
      ql[j][h][0] = pack_f16x2(v.x - f16_lo(qa[j][h][0]), v.y - f16_hi(qa[j][h][0]));
      ql[j][h][1] = pack_f16x2(v.z - f16_lo(qa[j][h][1]), v.w - f16_hi(qa[j][h][1]));
    }

  // ---- 1. scores of this warp's 16 keys: c[nt][0..1] = (head g, keys nt*8 + 2*tig, +1)
  float c[2][4];
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
    c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f;
#pragma unroll
    for (int j = 0; j < KJ; ++j) {
      mma_f16_16816(c[nt], qa[j][0][0], 0u, qa[j][0][1], 0u, kf[nt][j].x, kf[nt][j].y);
      mma_f16_16816(c[nt], qa[j][1][0], 0u, qa[j][1][1], 0u, kf[nt][j].z, kf[nt][j].w);
      mma_f16_16816(c[nt], ql[j][0][0], 0u, ql[j][0][1], 0u, kf[nt][j].x, kf[nt][j].y);
      mma_f16_16816(c[nt], ql[j][1][0], 0u, ql[j][1][1], 0u, kf[nt][j].z, kf[nt][j].w);
    }
  }
  // ---- 2. softmax statistics of head g over the warp's keys (quad reduction)
  float sv[4];
  float m = -INFINITY;
#pragma unroll
  for (int nt = 0; nt < 2; ++nt)
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int key = kw0 + nt * 8 + 2 * tig + e;
      sv[nt * 2 + e] = key < L ? c[nt][e] * scale : -INFINITY;
      m = fmaxf(m, sv[nt * 2 + e]);
    }
  m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
  m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
  float l = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    sv[i] = (m == -INFINITY) ? 0.f : __expf(sv[i] - m);
    l += sv[i];
  }
  l += __shfl_xor_sync(0xffffffffu, l, 1);
  l += __shfl_xor_sync(0xffffffffu, l, 2);
  if (g < GT) {
    if constexpr (!PVMMA) {
      *reinterpret_cast<float2*>(&ps[warp][g][2 * tig]) = make_float2(sv[0], sv[1]);
      *reinterpret_cast<float2*>(&ps[warp][g][8 + 2 * tig]) = make_float2(sv[2], sv[3]);
    }
    if (tig == 0) {
      mls[warp][g][0] = m;
      mls[warp][g][1] = l;
    }
  }
  __syncwarp();

  if constexpr (PVMMA) {
    // ---- 3. P.V on the tensor cores: A = probabilities of (head g; keys 2t, 2t+1 | 2t+8, 2t+9), hi + lo
    const uint32_t ph0 = pack_f16x2(sv[0], sv[1]), ph1 = pack_f16x2(sv[2], sv[3]);
    const uint32_t pl0 = pack_f16x2(sv[0] - f16_lo(ph0), sv[1] - f16_hi(ph0));
    const uint32_t pl1 = pack_f16x2(sv[2] - f16_lo(ph1), sv[3] - f16_hi(ph1));
#pragma unroll
    for (int j = 0; j < DH / 16; ++j) {
      uint32_t w[4];
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        const int i = j * 4 + q4;
        w[q4] = vr[i / (DPL / 2)][i % (DPL / 2)];
      }
      // even dims 16 j + 2 n and odd dims 16 j + 2 n + 1 as the two MMAs' columns n
      const uint32_t be0 = __byte_perm(w[0], w[1], 0x5410), be1 = __byte_perm(w[2], w[3], 0x5410);
      const uint32_t bo0 = __byte_perm(w[0], w[1], 0x7632), bo1 = __byte_perm(w[2], w[3], 0x7632);
      float ce[4] = {0.f, 0.f, 0.f, 0.f}, co[4] = {0.f, 0.f, 0.f, 0.f};
      mma_f16_16816(ce, ph0, 0u, ph1, 0u, be0, be1);
      mma_f16_16816(ce, pl0, 0u, pl1, 0u, be0, be1);
      mma_f16_16816(co, ph0, 0u, ph1, 0u, bo0, bo1);
      mma_f16_16816(co, pl0, 0u, pl1, 0u, bo0, bo1);
      // columns 2 tig, 2 tig + 1 of the two MMAs = dims 16 j + 4 tig .. + 3 of head g
      if (g < GT) *reinterpret_cast<float4*>(&red[warp][g][16 * j + 4 * tig]) = make_float4(ce[0], co[0], ce[1], co[1]);
    }
  }

  if constexpr (!PVMMA) {
  // ---- 3. P.V for the warp's 16 keys; lane owns dims [lane*DPL, +DPL)
  float acc[GT][DPL];
#pragma unroll
  for (int h = 0; h < GT; ++h)
#pragma unroll
    for (int d = 0; d < DPL; ++d) acc[h][d] = 0.f;
#pragma unroll
  for (int i4 = 0; i4 < 4; ++i4) {
    float4 pw[GT];
#pragma unroll
    for (int h = 0; h < GT; ++h) pw[h] = *reinterpret_cast<const float4*>(&ps[warp][h][i4 * 4]);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int i = i4 * 4 + e;
      float v[DPL];
      v[0] = f16_lo(vr[i][0]);
      v[1] = f16_hi(vr[i][0]);
      if (DPL == 4) {
        v[DPL - 2] = f16_lo(vr[i][DPL / 2 - 1]);
        v[DPL - 1] = f16_hi(vr[i][DPL / 2 - 1]);
      }
#pragma unroll
      for (int h = 0; h < GT; ++h) {
        const float w = e == 0 ? pw[h].x : (e == 1 ? pw[h].y : (e == 2 ? pw[h].z : pw[h].w));
#pragma unroll
        for (int d = 0; d < DPL; ++d) acc[h][d] += w * v[d];
      }
    }
  }
#pragma unroll
  for (int h = 0; h < GT; ++h)
#pragma unroll
    for (int d = 0; d < DPL; ++d) red[warp][h][lane * DPL + d] = acc[h][d];
  }
  __syncthreads();

  // ---- 4. merge the 4 warps, write the CTA partial.  The four rescaling factors of a head are computed once
  // (one thread per head) instead of once per output element: the element loop is then 4 FMAs and a store.
  const int stride = DH + 2;
  if (tid < GT) {
    const int h = tid;
    const float M = fmaxf(fmaxf(mls[0][h][0], mls[1][h][0]), fmaxf(mls[2][h][0], mls[3][h][0]));
    float ls = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float f = (mls[w][h][0] == -INFINITY) ? 0.f : __expf(mls[w][h][0] - M);
      mfac[h][w] = f;
      ls += f * mls[w][h][1];
    }
    float* dst = p.scratch + ((static_cast<size_t>(b) * p.n_q_heads + head0 + h) * p.n_splits + split) * stride;
    dst[DH] = M;
    dst[DH + 1] = ls;
  }
  __syncthreads();
  for (int idx = tid; idx < GT * DH; idx += kAttnThreads) {
    const int h = idx / DH, d = idx % DH;
    float o = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) o += mfac[h][w] * red[w][h][d];
    p.scratch[((static_cast<size_t>(b) * p.n_q_heads + head0 + h) * p.n_splits + split) * stride + d] = o;
  }
}

// Merge of the per-split partials of one (sequence, head) by log-sum-exp, in split order.
constexpr int kMaxSplits = 1024;
template <int DH>
__global__ void __launch_bounds__(DH) decode_attention_merge_kernel(const float* scratch, int n_q_heads, int n_splits,
                                                                    float* o, __nv_bfloat16* o_pack, int bp) {
  __shared__ float wgt[kMaxSplits];
  __shared__ float red_m[DH / 32], red_l[DH / 32];
  const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int stride = DH + 2;
  pdl_launch_dependents();
  pdl_wait();
  const float* base = scratch + (static_cast<size_t>(b) * n_q_heads + h) * n_splits * stride;
  // This thread's element of the first 32 partials, fetched before anything depends on anything: the statistics
  // below then cost no extra memory round trip (a 2048-key cache has 32 partials of 64 keys).
  constexpr int PRE = 32;
  float pre[PRE];
#pragma unroll
  for (int s = 0; s < PRE; ++s) pre[s] = s < n_splits ? __ldcg(base + s * stride + tid) : 0.f;
  float m = -INFINITY;
  for (int s = tid; s < n_splits; s += DH) {
    wgt[s] = __ldcg(base + s * stride + DH);
    m = fmaxf(m, wgt[s]);
  }
  m = warp_max(m);
  if (lane == 0) red_m[warp] = m;
  __syncthreads();
  float M = red_m[0];
#pragma unroll
  for (int w = 1; w < DH / 32; ++w) M = fmaxf(M, red_m[w]);
  float l = 0.f;
  for (int s = tid; s < n_splits; s += DH) {
    const float f = (wgt[s] == -INFINITY) ? 0.f : __expf(wgt[s] - M);
    wgt[s] = f;
    l += f * __ldcg(base + s * stride + DH + 1);
  }
  l = warp_sum(l);
  if (lane == 0) red_l[warp] = l;
  __syncthreads();
  float lsum = 0.f;
#pragma unroll
  for (int w = 0; w < DH / 32; ++w) lsum += red_l[w];
  float acc = 0.f;
#pragma unroll
  for (int s = 0; s < PRE; ++s)
    if (s < n_splits) acc += wgt[s] * pre[s];
#pragma unroll 8
  for (int s = PRE; s < n_splits; ++s) acc += wgt[s] * __ldcg(base + s * stride + tid);
  const float val = lsum > 0.f ? acc / lsum : 0.f;
  o[(static_cast<size_t>(b) * n_q_heads + h) * DH + tid] = val;
  if (o_pack) {  // the output projection's staged operand: hi part in row b, lo part in row bp + b
    const size_t K = static_cast<size_t>(n_q_heads) * DH, col = static_cast<size_t>(h) * DH + tid;
    const __nv_bfloat16 hi = __float2bfloat16_rn(val);
    o_pack[b * K + col] = hi;
    o_pack[(bp + b) * K + col] = __float2bfloat16_rn(val - __bfloat162float(hi));
    if (b == static_cast<int>(gridDim.y) - 1)  // the last sequence's CTAs also clear the padding rows
      for (int r = b + 1; r < bp; ++r) o_pack[r * K + col] = o_pack[(bp + r) * K + col] = __float2bfloat16_rn(0.f);
  }
}

cudaLaunchConfig_t make_cfg(dim3 grid, dim3 block, cudaStream_t stream, bool pdl, cudaLaunchAttribute* at) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.stream = stream;
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  return cfg;
}

template <int GT>
cudaError_t launch_gt(const DecodeAttnParams& p, cudaStream_t stream, bool pdl) {
  cudaLaunchAttribute at[1];
  cudaLaunchConfig_t cfg = make_cfg(dim3(p.n_splits, p.n_q_heads / GT, p.batch), dim3(kAttnThreads), stream, pdl, at);
  if (p.batch > 8) {  // throughput regime: P.V on the tensor cores
    if (p.head_dim == 128) return cudaLaunchKernelEx(&cfg, decode_attention_kernel<GT, 128, true>, p);
    return cudaLaunchKernelEx(&cfg, decode_attention_kernel<GT, 64, true>, p);
  }
  if (p.head_dim == 128) return cudaLaunchKernelEx(&cfg, decode_attention_kernel<GT, 128, false>, p);
  return cudaLaunchKernelEx(&cfg, decode_attention_kernel<GT, 64, false>, p);
}

int heads_per_cta(int n_q_heads, int n_kv_heads) {
  const int group = n_q_heads / n_kv_heads;
  int gt = 1;
  while (gt < 8 && group % (gt * 2) == 0) gt *= 2;
  return gt;
}

}  // namespace

int decode_attention_splits(int batch, int n_kv_heads, int max_len, int sm_count) {
  (void)batch, (void)n_kv_heads, (void)sm_count;
  const int n = (max_len + kChunk - 1) / kChunk;  // one CTA per 64 keys
  return n < 1 ? 1 : n;
}

// scratch: [batch][Hq][n_splits][Dh + 2] floats (o, m, l per split)
size_t decode_attention_scratch_floats(int batch, int n_q_heads, int head_dim, int n_splits) {
  return static_cast<size_t>(batch) * n_q_heads * n_splits * (head_dim + 2);
}

static int g_attn_impl = 0;
void set_decode_attention_impl(int impl) { g_attn_impl = impl == 1 || impl == 2 ? impl : 0; }

cudaError_t launch_decode_attention(const DecodeAttnParams& p, cudaStream_t stream, bool pdl) {
  if (p.n_splits * kChunk < p.max_len || p.n_splits > kMaxSplits) return cudaErrorInvalidValue;
  cudaError_t e;
  int n_partials = p.n_splits;  // partials per (sequence, head) the merge reads
  // Throughput regime: the TMA-fed tcgen05 kernel, one partial per 128 keys (the scratch is sized for one per 64).
  // Only where there is enough to stream: it cannot share an SM with the GEMM before or after it (217 KB of shared
  // memory), so below ~2000 tiles its start-up costs more than its bandwidth gains (measured inside decode steps:
  // TP-rank slice batch 64, 1088 tiles, +4 %; 70B shape batch 32 / 64, 3072 / 6144 tiles, -0.7 % / -1.7 %).
  const long tiles128 = static_cast<long>(p.batch) * p.n_kv_heads * ((p.max_len + 127) / 128);
  if (p.batch > 8 && (g_attn_impl == 2 || (g_attn_impl == 0 && tiles128 >= 2048)) && decode_attention_tc_usable(p)) {
    n_partials = p.max_len > 128 ? (p.max_len + 127) / 128 : 1;
    e = launch_decode_attention_tc(p, n_partials, p.status, stream, pdl);
  } else {
    switch (heads_per_cta(p.n_q_heads, p.n_kv_heads)) {
      case 8: e = launch_gt<8>(p, stream, pdl); break;
      case 4: e = launch_gt<4>(p, stream, pdl); break;
      case 2: e = launch_gt<2>(p, stream, pdl); break;
      default: e = launch_gt<1>(p, stream, pdl); break;
    }
  }
  if (e != cudaSuccess) return e;
  cudaLaunchAttribute at[1];
  cudaLaunchConfig_t cfg = make_cfg(dim3(p.n_q_heads, p.batch), dim3(p.head_dim), stream, pdl, at);
  const float* scratch = p.scratch;
  __nv_bfloat16* o_pack = p.o_pack;
  const int bp = p.o_pack_bp;
  if (o_pack && bp < p.batch) return cudaErrorInvalidValue;
  if (p.head_dim == 128)
    return cudaLaunchKernelEx(&cfg, decode_attention_merge_kernel<128>, scratch, p.n_q_heads, n_partials, p.o, o_pack, bp);
  return cudaLaunchKernelEx(&cfg, decode_attention_merge_kernel<64>, scratch, p.n_q_heads, n_partials, p.o, o_pack, bp);
}

}  // namespace ladder

// ---------------------------------------------------------------------------------------------
// Allocation-free variant of the decode-attention entry point.
//
// Some hosts of this library may not allocate device memory at all once they are running: an
// inference server that has handed every byte of the device to its own pool allocator, a process
// inside a memory-capped container slice, code running under a framework that forbids cudaMalloc
// after start-up.  For them the per-split partial results (the only scratch this kernel needs) live
// in a fixed array inside the library image instead of a caller buffer.  The array is part of every
// context that loads the library and stays resident until the process exits, hence the modest cap.
namespace ladder {
namespace {

constexpr size_t kNoAllocScratchFloats = size_t(2) << 20;  // 8 MiB: e.g. batch 4, 64 heads x 128, 2048 keys
static __device__ __align__(256) float g_noalloc_scratch[kNoAllocScratchFloats];

constexpr int kMaxDevices = 64;
float* g_noalloc_ptr[kMaxDevices];  // device address of the array on each device, resolved once

// In host code the array's name is only a handle for the runtime; the address a kernel can use
// must be looked up per device, with that device current.
cudaError_t noalloc_scratch(float** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!g_noalloc_ptr[dev]) {
    float* ptr = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    g_noalloc_ptr[dev] = ptr;
  }
  *out = g_noalloc_ptr[dev];
  return cudaSuccess;
}

}  // namespace
}  // namespace ladder

extern "C" ladder_status_t ladder_op_decode_attention_noalloc(const float* q, const void* k, const void* v,
                                                              const int32_t* kv_len, int32_t batch, int32_t n_q_heads,
                                                              int32_t n_kv_heads, int32_t head_dim,
                                                              int32_t max_seq_len, void* o, void* cuda_stream) {
  using namespace ladder;
  if (!q || !k || !v || !kv_len || !o) return LADDER_ERR_INVALID_ARG;
  if (batch < 1 || n_kv_heads < 1 || n_q_heads < 1 || n_q_heads % n_kv_heads || (head_dim != 64 && head_dim != 128) ||
      max_seq_len < 1)
    return LADDER_ERR_INVALID_ARG;
  if (decode_attention_misaligned(q, k, v, o, nullptr, kv_len)) return LADDER_ERR_INVALID_ARG;
  if (max_seq_len > kDecodeAttnMaxKeys) return LADDER_ERR_UNSUPPORTED;
  const int n_splits = decode_attention_splits(batch, n_kv_heads, max_seq_len, 0);
  if (decode_attention_scratch_floats(batch, n_q_heads, head_dim, n_splits) > kNoAllocScratchFloats)
    return LADDER_ERR_UNSUPPORTED;  // batch * heads * ceil(max_seq_len / 64) * (head_dim + 2) floats exceed 8 MiB
  float* scratch = nullptr;
  if (noalloc_scratch(&scratch) != cudaSuccess) return LADDER_ERR_CUDA;
  DecodeAttnParams a = {};
  a.q = q;
  a.k = static_cast<const kv_t*>(k);
  a.v = static_cast<const kv_t*>(v);
  a.kv_len = kv_len;
  a.kv_len_offset = 0;
  a.batch = batch;
  a.n_q_heads = n_q_heads;
  a.n_kv_heads = n_kv_heads;
  a.head_dim = head_dim;
  a.max_seq_len = max_seq_len;
  a.max_len = max_seq_len;
  a.n_splits = n_splits;
  a.scratch = scratch;  // every split writes its whole partial before the merge reads it: nothing to clear
  a.o = static_cast<float*>(o);
  return launch_decode_attention(a, static_cast<cudaStream_t>(cuda_stream), false) == cudaSuccess ? LADDER_OK
                                                                                                   : LADDER_ERR_CUDA;
}

