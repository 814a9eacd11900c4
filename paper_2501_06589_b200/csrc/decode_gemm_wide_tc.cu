// Weight-streaming decode GEMM for batch 9..64 on the 5th-generation tensor cores (tcgen05 / UMMA):
//   acc[b, n] = sum_k act[b, k] * W[n, k]          W bf16 [N, K], act fp32 [batch, K]
// "Swapped" operands: a tile of 128 weight rows is the M side of the MMA (A operand, straight from
// shared memory), the batch is the N side.  The activations are split into a bf16 high and low part
// (x ~ hi + lo) that sit side by side as 2 x Bp MMA columns (Bp = batch padded to 16 / 32 / 64), so
// the extra precision costs no extra instruction; their sum is formed in the epilogue.
//
// Two kernels per GEMM:
//   1. wide_stage_kernel: fp32 activations (x gain for RMSNorm) -> bf16 [2 Bp, K] in scratch, sums of squares
//      per 2048-wide K slice (the GEMM adds them in slice order: deterministic).
//   2. decode_gemm_wide_tc_kernel: persistent CTAs, one per SM, three roles that meet at mbarriers:
//        warp 0     TMA producer: per 64-wide K block one [128 rows x 64] box of W (L2 evict-first) and
//                   one [2 Bp x 64] box of the staged activations (L2-resident), 128-byte swizzle, into a
//                   6..10-stage ring (20..32 KB per stage, ~100-160 KB of weights in flight per SM);
//        warp 1     MMA issuer: tcgen05.mma M 128, N 2 Bp, K 16, kind::f16, fp32 accumulators in tensor
//                   memory (two buffers, so the epilogue of one segment overlaps the MMAs of the next);
//        warps 2-9  epilogue: tcgen05.ld (a thread owns one weight row and half of the batch columns), hi + lo,
//                   1/rms, then residual add (Eq. 1 / Eq. 2) / SwiGLU / rotary + KV append / plain store.
// Work split: the T row tiles x nkb K blocks are cut into one contiguous range per CTA (equal to within
// one K block), so every SM streams the same number of bytes whatever N and K are.  A tile whose K
// range is shared by several CTAs is finished by the one that arrives last: every piece goes to an
// L2-resident scratch, a ticket per tile counts arrivals, and the last CTA adds the pieces in CTA order
// (deterministic) and runs the epilogue.
// Every wait is bounded; on a protocol error the kernel records it, drains and frees its TMEM.
#include <cuda.h>

#include "common.cuh"
#include "kernels.h"

namespace ladder {
namespace {

constexpr int BM = 128, BK = 64, UMMA_K = 16;
constexpr int W_BYTES = BM * BK * 2;  // 16 KB
constexpr int kWideThreads = 320;   // TMA producer warp, MMA warp, 8 epilogue warps
constexpr int kWideMaxTiles = 2048;   // tickets
constexpr int kWideMaxCtas = 160;     // partial slots

template <int NP>
struct WCfg {
  static constexpr int BP = NP / 2;
  static constexpr int ACT_BYTES = NP * BK * 2;
  static constexpr int STAGE_BYTES = W_BYTES + ACT_BYTES;
  static constexpr int STAGES = (200 * 1024) / STAGE_BYTES;
  static constexpr int OFF_BARS = STAGES * STAGE_BYTES;  // full[], empty[], tmem_full[2], tmem_empty[2], tmem slot, flag
  static constexpr int SMEM = OFF_BARS + (2 * STAGES + 4) * 8 + 64 + 2 * 64 * 4 + 1024;
  static constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(NP >> 3) << 17) |
                                    (static_cast<uint32_t>(BM >> 4) << 24);
  static_assert(SMEM <= 232448, "shared memory budget");
};

struct WideArgs {
  SmallMParams p;
  int bp;                  // padded batch
  int tiles, nkb;          // row tiles, K blocks
  const float* ssq;        // [bp][n_slices] sums of squares per K slice (ACT_F32_NORM)
  int n_slices;
  float* partial;          // [grid][2][bp][128]
  int32_t* tickets;        // [tiles], zero between launches
  WidePeer wp;             // push_channel != 0: the output goes to the peers' receive slots
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
          smem_u32(dst)),
      "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d_hint(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar,
                                                 uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], "
      "[%2], %5;" ::"r"(smem_u32(dst)),
      "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_ld8(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tc_ld4(uint32_t taddr, uint32_t (&r)[4]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tc_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand tile of rows x 64 bf16, 128-byte swizzle
// (rows of 128 bytes, 8-row swizzle atoms of 1024 bytes), tile base 1024-byte aligned.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}

// ---------------------------------------------------------------- activation staging
// One CTA per (padded batch row, 2048-wide K slice): y = x (* gain), hi = bf16(y), lo = bf16(y - hi); rows
// >= batch are zero.  The slice's sum of squares goes to ssq[row][slice]; the GEMM adds the slices in order.
constexpr int kStageSlice = 2048;
// A pending that is pulled (tensor parallelism over peer memory): the sum over the ranks, in rank order, of this rank's
// receive slots [channel][turn & 1][0 .. world).  Every element there is a (value, sequence number) pair written by
// one 8-byte store of the rank that produced it; an element has arrived when its number is turn + 1.
struct StagePull {
  PeerView peer;
  int channel[2];  // channel + 1 of pending / pending2, 0 = not pulled
  int32_t* status;
};

// y[0 .. 8) += the eight values at element offset `off` of every rank's slot.  Polls (bounded) until they are there;
// false if the wait ran out.
__device__ __forceinline__ bool pull_add8(const StagePull& pl, int ch, uint32_t turn, size_t off, float (&y)[8]) {
  unsigned char* base = pl.peer.base[pl.peer.rank];
  const uint32_t seq = turn + 1u;
  bool ok = true;
  for (int r = 0; r < pl.peer.world && ok; ++r) {
    const uint4* src = reinterpret_cast<const uint4*>(
        reinterpret_cast<const uint2*>(peer_slot(base, pl.peer.world, pl.peer.max_floats, ch, turn & 1u, r)) + off);
    uint4 v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = peer_ld_pairs(src + i);
    auto there = [&] {
      bool t = true;
#pragma unroll
      for (int i = 0; i < 4; ++i) t = t && v[i].y == seq && v[i].w == seq;
      return t;
    };
    if (!there()) {  // bounded by the SM's cycle counter (~0.3 s); no waiting at all once a wait has run out anywhere
      const long long t0 = clock64();
      const volatile int32_t* st = pl.status;
      if (st && (*st & LADDER_DEV_TIMEOUT)) ok = false;
      for (uint32_t it = 1; ok && !there(); ++it) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (v[i].y != seq || v[i].w != seq) v[i] = peer_ld_pairs(src + i);
        if ((it & 255u) == 0 && (clock64() - t0 > kWaitCycles || (st && (*st & LADDER_DEV_TIMEOUT)))) ok = false;
      }
    }
    if (ok) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        y[2 * i] += __uint_as_float(v[i].x);
        y[2 * i + 1] += __uint_as_float(v[i].z);
      }
    }
  }
  return ok;
}

__global__ void __launch_bounds__(256) wide_stage_kernel(const float* x, const __nv_bfloat16* gain, int norm, int batch,
                                                         int bp, int K, __nv_bfloat16* stage, float* ssq_out,
                                                         const float* pending, const float* pending2,
                                                         float* sum_out, const StagePull pl) {
  __shared__ float red[8];
  const int b = blockIdx.x, slice = blockIdx.y, tid = threadIdx.x;
  pdl_launch_dependents();
  pdl_wait();
  const bool pulls = pl.peer.world > 0 && (pl.channel[0] | pl.channel[1]);
  uint32_t turn0 = 0, turn1 = 0;
  if (pulls) {  // the exchanges consumed so far on the pulled channels: receive-slot parity and sequence number
    PeerHeader* hdr = peer_header(pl.peer.base[pl.peer.rank]);
    if (pl.channel[0]) turn0 = *reinterpret_cast<volatile uint32_t*>(&hdr->turn[pl.channel[0] - 1]);
    if (pl.channel[1]) turn1 = *reinterpret_cast<volatile uint32_t*>(&hdr->turn[pl.channel[1] - 1]);
    pending = pl.channel[0] ? nullptr : pending;  // a pulled pending has no plain buffer
    pending2 = pl.channel[1] ? nullptr : pending2;
  }
  bool pull_ok = true;
  __nv_bfloat16* hi = stage + static_cast<size_t>(b) * K;
  __nv_bfloat16* lo = stage + static_cast<size_t>(bp + b) * K;
  float ssq = 0.f;
  const int k = slice * kStageSlice + tid * 8;
  if (k < K) {
    float y[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (b < batch) {
      const float4 a = __ldcg(reinterpret_cast<const float4*>(x + static_cast<size_t>(b) * K + k));
      const float4 c = __ldcg(reinterpret_cast<const float4*>(x + static_cast<size_t>(b) * K + k + 4));
      y[0] = a.x, y[1] = a.y, y[2] = a.z, y[3] = a.w, y[4] = c.x, y[5] = c.y, y[6] = c.z, y[7] = c.w;
      if (pulls && pl.channel[0])  // ... the module output summed over the tensor-parallel ranks
        pull_ok = pull_add8(pl, pl.channel[0] - 1, turn0, static_cast<size_t>(b) * K + k, y) && pull_ok;
      if (pending) {  // x_m = x_{m-1} + (the module output stored by an earlier GEMM)
        const float4 pa = __ldcg(reinterpret_cast<const float4*>(pending + static_cast<size_t>(b) * K + k));
        const float4 pc = __ldcg(reinterpret_cast<const float4*>(pending + static_cast<size_t>(b) * K + k + 4));
        y[0] += pa.x, y[1] += pa.y, y[2] += pa.z, y[3] += pa.w, y[4] += pc.x, y[5] += pc.y, y[6] += pc.z, y[7] += pc.w;
      }
      if (pulls && pl.channel[1])
        pull_ok = pull_add8(pl, pl.channel[1] - 1, turn1, static_cast<size_t>(b) * K + k, y) && pull_ok;
      if (pending2) {  // ... and the one after it
        const float4 pa = __ldcg(reinterpret_cast<const float4*>(pending2 + static_cast<size_t>(b) * K + k));
        const float4 pc = __ldcg(reinterpret_cast<const float4*>(pending2 + static_cast<size_t>(b) * K + k + 4));
        y[0] += pa.x, y[1] += pa.y, y[2] += pa.z, y[3] += pa.w, y[4] += pc.x, y[5] += pc.y, y[6] += pc.z, y[7] += pc.w;
      }
      if (sum_out) {
        *reinterpret_cast<float4*>(sum_out + static_cast<size_t>(b) * K + k) = make_float4(y[0], y[1], y[2], y[3]);
        *reinterpret_cast<float4*>(sum_out + static_cast<size_t>(b) * K + k + 4) = make_float4(y[4], y[5], y[6], y[7]);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) ssq += y[i] * y[i];
      if (norm) {
        const uint4 g = __ldg(reinterpret_cast<const uint4*>(gain + k));
        y[0] *= bf16_lo(g.x), y[1] *= bf16_hi(g.x), y[2] *= bf16_lo(g.y), y[3] *= bf16_hi(g.y);
        y[4] *= bf16_lo(g.z), y[5] *= bf16_hi(g.z), y[6] *= bf16_lo(g.w), y[7] *= bf16_hi(g.w);
      }
    }
    uint4 h, l;
    h.x = pack_bf16x2(y[0], y[1]), h.y = pack_bf16x2(y[2], y[3]), h.z = pack_bf16x2(y[4], y[5]), h.w = pack_bf16x2(y[6], y[7]);
    l.x = pack_bf16x2(y[0] - bf16_lo(h.x), y[1] - bf16_hi(h.x));
    l.y = pack_bf16x2(y[2] - bf16_lo(h.y), y[3] - bf16_hi(h.y));
    l.z = pack_bf16x2(y[4] - bf16_lo(h.z), y[5] - bf16_hi(h.z));
    l.w = pack_bf16x2(y[6] - bf16_lo(h.w), y[7] - bf16_hi(h.w));
    *reinterpret_cast<uint4*>(hi + k) = h;
    *reinterpret_cast<uint4*>(lo + k) = l;
  }
  if (!pull_ok && pl.status) atomicOr(pl.status, LADDER_DEV_TIMEOUT);
  ssq = warp_sum(ssq);
  if ((tid & 31) == 0) red[tid >> 5] = ssq;
  __syncthreads();
  if (tid == 0) {
    float t = 0.f;
    for (int w = 0; w < 8; ++w) t += red[w];
    ssq_out[b * gridDim.y + slice] = t;
    if (pulls) {  // the last CTA of the launch moves the pulled channels on (their other receive slot is next)
      PeerHeader* hdr = peer_header(pl.peer.base[pl.peer.rank]);
      const int first = (pl.channel[0] ? pl.channel[0] : pl.channel[1]) - 1;
      __threadfence();
      if (atomicAdd(&hdr->ticket[first], 1u) == gridDim.x * gridDim.y - 1) {
        hdr->ticket[first] = 0;
        for (int i = 0; i < 2; ++i)
          if (pl.channel[i]) hdr->turn[pl.channel[i] - 1] += 1u;
        __threadfence();
      }
    }
  }
}

// ---------------------------------------------------------------- epilogue of one weight row
// A thread owns weight row n and CB batch columns b0 .. b0 + CB - 1.  Lanes of a warp hold consecutive rows, so
// the (gate, up) and rotary pairs are neighbouring lanes; all lanes take part in the shuffles.
// Everything the tail reads from global memory (the residual addend, the rotary factors) is fetched by
// epi_prefetch for all CB columns at once, ahead of the accumulators or pieces: a load placed after a store to
// memory that may alias cannot be moved ahead of it by the compiler, and one dependent L2 round trip per
// column cost 20 us per launch at batch 64.  pa = addend (EPI_RESID) or cos, pb = sin (EPI_QKV_ROPE).
// pos_s[b] = position of batch row b (-1 for b >= batch), read once per CTA.
template <int CB>
__device__ __forceinline__ void epi_prefetch(const SmallMParams& p, int n, int b0, int lane, const int* pos_s,
                                             float (&pa)[CB], float (&pb)[CB]) {
  const bool row_ok = n < p.N;
  if (p.epi_mode == EPI_RESID) {
#pragma unroll
    for (int j = 0; j < CB; ++j)
      pa[j] = (b0 + j < p.batch && row_ok) ? __ldcg(p.addend + static_cast<size_t>(b0 + j) * p.N + n) : 0.f;
  } else if (p.epi_mode == EPI_QKV_ROPE) {
    const QkvEpilogue& e = p.qkv;
    const int Dh = e.head_dim;
    const bool rotated = !(lane & 1) && row_ok && n < (e.n_q_heads + e.n_kv_heads) * Dh;
#pragma unroll
    for (int j = 0; j < CB; ++j) {
      const int pos = pos_s[b0 + j];
      const float2 cs = (rotated && pos >= 0 && pos < e.max_seq_len)
                            ? __ldg(e.rope + static_cast<size_t>(pos) * (Dh >> 1) + ((n % Dh) >> 1))
                            : make_float2(1.f, 0.f);
      pa[j] = cs.x;
      pb[j] = cs.y;
    }
  }
}

// v[j] = finished accumulator of row n and batch row b0 + j.
template <int CB, bool PUSH>
__device__ __forceinline__ void epi_apply(const SmallMParams& p, int n, int b0, float (&v)[CB], int lane,
                                          const int* pos_s, const float (&pa)[CB], const float (&pb)[CB], int bp,
                                          const WidePeer& wp, const size_t* push_s) {
  const bool row_ok = n < p.N;
  if (PUSH) {
    // tensor parallelism over peer memory (EPI_PLAIN, or EPI_RESID with a local addend): this rank's partial sum goes straight into its receive
    // slot on every rank, every value with the exchange's sequence number in one 8-byte store (lanes hold
    // consecutive rows: 256-byte segments per batch row and peer)
    const size_t off = push_s[0];
    const uint32_t seq = static_cast<uint32_t>(push_s[1]);
#pragma unroll 1
    for (int w = 0; w < wp.peer.world; ++w) {
      uint2* out = reinterpret_cast<uint2*>(reinterpret_cast<float*>(wp.peer.base[w] + kPeerHeaderBytes) + off);
#pragma unroll
      for (int j = 0; j < CB; ++j) {
        const int b = b0 + j;
        if (b < p.batch && row_ok)
          peer_st_pair(out + static_cast<size_t>(b) * p.N + n, p.epi_mode == EPI_RESID ? v[j] + pa[j] : v[j], seq);
      }
    }
  } else if (p.epi_mode == EPI_RESID || p.epi_mode == EPI_PLAIN) {
    float* out = static_cast<float*>(p.out);
#pragma unroll
    for (int j = 0; j < CB; ++j) {
      const int b = b0 + j;
      if (b < p.batch && row_ok) out[static_cast<size_t>(b) * p.N + n] = p.epi_mode == EPI_RESID ? v[j] + pa[j] : v[j];
    }
  } else if (p.epi_mode == EPI_SWIGLU) {
    float* out = static_cast<float*>(p.out);
#pragma unroll
    for (int j = 0; j < CB; ++j) {
      const int b = b0 + j;
      const float up = __shfl_down_sync(0xffffffffu, v[j], 1);
      if (!(lane & 1) && row_ok) {
        const float gt = v[j];
        const float hv = b < p.batch ? gt / (1.f + __expf(-gt)) * up : 0.f;
        if (b < p.batch) out[static_cast<size_t>(b) * (p.N >> 1) + (n >> 1)] = hv;
        if (p.wide_pack_out) {  // the down projection's staged operand (padding rows written as zero)
          const size_t kc = static_cast<size_t>(p.N >> 1), col = static_cast<size_t>(n >> 1);
          const __nv_bfloat16 hi = __float2bfloat16_rn(hv);
          p.wide_pack_out[b * kc + col] = hi;
          p.wide_pack_out[(bp + b) * kc + col] = __float2bfloat16_rn(hv - __bfloat162float(hi));
        }
      }
    }
  } else if (p.epi_mode == EPI_QKV_ROPE) {
    const QkvEpilogue& e = p.qkv;
    const int Dh = e.head_dim, nq = e.n_q_heads * Dh, nk = e.n_kv_heads * Dh;
#pragma unroll
    for (int j = 0; j < CB; ++j) {
      const int b = b0 + j;
      float v0 = v[j], v1 = __shfl_down_sync(0xffffffffu, v[j], 1);
      if ((lane & 1) || b >= p.batch || !row_ok) continue;
      const int pos = pos_s[b];
      if (pos < 0 || pos >= e.max_seq_len) {
        if (p.status) atomicOr(p.status, LADDER_DEV_CACHE_OVERFLOW);
        continue;
      }
      if (n < nq + nk) {
        const float a0 = v0 * pa[j] - v1 * pb[j], a1 = v0 * pb[j] + v1 * pa[j];
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

// barrier among the 256 epilogue threads that also ANDs a predicate, so that they leave together
__device__ __forceinline__ bool epi_bar_and(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 p, %1, 0;\n\t"
      "bar.red.and.pred q, 1, 256, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r)
      : "r"(static_cast<uint32_t>(pred))
      : "memory");
  return r != 0;
}

// contiguous split of `total` K-block-tiles over `grid` CTAs: the first `rem` CTAs get one more
struct Split {
  int per, rem;
  __device__ __forceinline__ int start(int c) const { return c * per + min(c, rem); }
  __device__ __forceinline__ int owner(int x) const {
    const int big = rem * (per + 1);
    return x < big ? x / (per + 1) : rem + (x - big) / per;
  }
};

template <int NP, bool PUSH>
__global__ void __launch_bounds__(kWideThreads, 1)
decode_gemm_wide_tc_kernel(const WideArgs a, const __grid_constant__ CUtensorMap map_w,
                           const __grid_constant__ CUtensorMap map_act) {
  using C = WCfg<NP>;
  constexpr int BP = C::BP, STAGES = C::STAGES;
  constexpr int HALVES = BP >= 16 ? 2 : 1;  // the batch columns are split between two sets of four epilogue warps
  constexpr int CPH = BP / HALVES;
  constexpr int CB = CPH < 16 ? CPH : 16;   // batch columns handled per epilogue pass
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + C::OFF_BARS);
  uint64_t* empty = full + STAGES;
  uint64_t* tmem_full = empty + STAGES;
  uint64_t* tmem_empty = tmem_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + 2);
  volatile int* last_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  size_t* push_s = reinterpret_cast<size_t*>(tmem_slot + 2);  // float offset of the receive slot pushed into; sequence number
  float* rstd_s = reinterpret_cast<float*>(smem + C::OFF_BARS + (2 * STAGES + 4) * 8 + 64);  // [BP] 1/rms
  int* pos_s = reinterpret_cast<int*>(rstd_s + 64);                                            // [BP] positions

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const SmallMParams& p = a.p;
  const int nkb = a.nkb;
  const int total = a.tiles * nkb;
  const Split sp = {total / static_cast<int>(gridDim.x), total % static_cast<int>(gridDim.x)};
  const int my_start = sp.start(blockIdx.x), my_end = sp.start(blockIdx.x + 1);

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&tmem_full[b], 1);
      mbar_init(&tmem_empty[b], 8);
    }
    fence_barrier_init();
  }
  if (warp == 1) {  // TMEM: two accumulators of NP fp32 columns x 128 lanes
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "n"(2 * NP < 32 ? 32 : 2 * NP)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_launch_dependents();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_slot);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const uint64_t pol = l2_policy_evict_first();
      bool ok = true;
      const int n_it = my_end - my_start;
      // First ring fill: the weight boxes of up to STAGES K blocks go out before the wait on the kernel that
      // staged the activations (weights depend on nothing), their activation boxes right after it.
      const int pre = n_it < STAGES ? n_it : STAGES;
      for (int i = 0; i < pre; ++i) {
        const int pos = my_start + i, t = pos / nkb, kb = pos - t * nkb;
        mbar_expect_tx(&full[i], C::STAGE_BYTES);
        tma_load_2d_hint(smem + i * C::STAGE_BYTES, &map_w, kb * BK, t * BM, &full[i], pol);
      }
      pdl_wait();
      for (int i = 0; i < pre; ++i) {
        const int pos = my_start + i, kb = pos % nkb;
        tma_load_2d(smem + i * C::STAGE_BYTES + W_BYTES, &map_act, kb * BK, 0, &full[i]);
      }
      int it = pre;
      for (; it < n_it; ++it) {
        const int s = it % STAGES;
        ok = mbar_wait_bounded(&empty[s], ((it / STAGES) & 1) ^ 1u);
        if (!ok) break;
        const int pos = my_start + it, t = pos / nkb, kb = pos - t * nkb;
        uint8_t* st = smem + s * C::STAGE_BYTES;
        mbar_expect_tx(&full[s], C::STAGE_BYTES);
        tma_load_2d_hint(st, &map_w, kb * BK, t * BM, &full[s], pol);
        tma_load_2d(st + W_BYTES, &map_act, kb * BK, 0, &full[s]);
      }
      if (!ok) {
        if (p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
        for (int j = 1; j <= STAGES && j <= it; ++j) {  // wait (bounded) for the copies still in flight
          const int i2 = it - j;
          mbar_wait_bounded(&full[i2 % STAGES], (i2 / STAGES) & 1);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = true;
      int it = 0, seg = 0;
      for (int pos = my_start; pos < my_end && ok; ++seg) {
        const int t = pos / nkb, kb0 = pos - t * nkb, kb1 = min(nkb, kb0 + (my_end - pos));
        const int ab = seg & 1;
        ok = mbar_wait_bounded(&tmem_empty[ab], ((seg >> 1) & 1) ^ 1u);  // the epilogue has drained this accumulator
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + ab * NP;
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % STAGES;
          ok = mbar_wait_bounded(&full[s], (it / STAGES) & 1);
          if (!ok) break;
          tc_fence_after();
          const uint32_t w_addr = smem_u32(smem + s * C::STAGE_BYTES);
          const uint64_t dw = smem_desc(w_addr), dact = smem_desc(w_addr + W_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)  // +32 bytes along K inside the swizzled row = +2 in the address field
            tc_mma(d_tmem, dw + 2 * k, dact + 2 * k, C::IDESC, (kb > kb0 || k > 0) ? 1u : 0u);
          tc_commit(&empty[s]);  // the stage is free once these MMAs have read it
        }
        if (ok) tc_commit(&tmem_full[ab]);
        pos += kb1 - kb0;
      }
      if (!ok && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;          // the TMEM lane quarter this warp may access
    const int half = (warp - 2) >> 2;  // which share of the batch columns
    const int et = tid - 64;         // 0..255
    const int r = q * 32 + lane;     // row inside the tile
    const int c_begin = half < HALVES ? half * CPH : 0, c_end = half < HALVES ? c_begin + CPH : 0;
    bool ok = true;
    int seg = 0;
    pdl_wait();  // the sums of squares, the positions, the addend and the destination belong to earlier kernels
    if (et < BP) {   // 1/rms of every batch row: the K slices' sums of squares added in slice order
      float t = 0.f;
      if (p.act_mode == ACT_F32_NORM)
        for (int sl = 0; sl < a.n_slices; ++sl) t += a.ssq[et * a.n_slices + sl];
      rstd_s[et] = p.act_mode == ACT_F32_NORM ? rsqrtf(t / static_cast<float>(p.K) + p.eps) : 1.f;
    } else if (et >= 128 && et - 128 < BP) {
      const int b = et - 128;
      pos_s[b] = (p.epi_mode == EPI_QKV_ROPE && b < p.batch) ? p.qkv.seq_lens[b] : -1;
    }
    // receive-slot parity of this exchange: the channel was last moved on by a staging launch that lies before
    // this kernel's predecessors in stream order
    if (PUSH && et == 255) {  // receive slot [channel][turn & 1][this rank]: the same offset on every rank
      // (the channel was last moved on by a staging launch that lies before this kernel's predecessors in stream order)
      const int ch = a.wp.push_channel - 1;
      const uint32_t turn = *reinterpret_cast<volatile uint32_t*>(&peer_header(a.wp.peer.base[a.wp.peer.rank])->turn[ch]);
      push_s[0] = ((static_cast<size_t>(ch) * 2 + (turn & 1u)) * a.wp.peer.world + a.wp.peer.rank) * (2 * a.wp.peer.max_floats);
      push_s[1] = turn + 1u;
    }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    for (int pos = my_start; pos < my_end; ++seg) {
      const int t = pos / nkb, kb0 = pos - t * nkb, kb1 = min(nkb, kb0 + (my_end - pos));
      pos += kb1 - kb0;
      const int ab = seg & 1;
      const bool whole = kb0 == 0 && kb1 == nkb;
      const int n = t * BM + r;
      ok = epi_bar_and(ok && mbar_wait_bounded(&tmem_full[ab], (seg >> 1) & 1));  // all eight warps agree
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + ab * NP;
      // where this CTA's piece of a shared tile goes: slot 0 if the tile is the first of its range, else slot 1
      const int my_slot = (t == my_start / nkb) ? 0 : 1;
      // piece layout: [TMEM lane quarter][group of 4 batch columns][lane] float4, so that a warp's store and
      // the last arrival's load of one column group are 512 contiguous bytes
      float4* piece = reinterpret_cast<float4*>(a.partial + (static_cast<size_t>(blockIdx.x) * 2 + my_slot) * BP * BM) +
                      q * (BP / 4) * 32 + lane;
#pragma unroll 1
      for (int b0 = c_begin; b0 < c_end; b0 += CB) {
        float v[CB], pa[CB], pb[CB];
        if (whole) epi_prefetch<CB>(p, n, b0, lane, pos_s, pa, pb);
        if constexpr (CB == 4) {
          uint32_t h[4], l[4];
          tc_ld4(taddr + b0, h);
          tc_ld4(taddr + BP + b0, l);
          tc_ld_wait();
#pragma unroll
          for (int j = 0; j < 4; ++j) v[j] = __uint_as_float(h[j]) + __uint_as_float(l[j]);
        } else if constexpr (CB == 8) {
          uint32_t h[8], l[8];
          tc_ld8(taddr + b0, h);
          tc_ld8(taddr + BP + b0, l);
          tc_ld_wait();
#pragma unroll
          for (int j = 0; j < 8; ++j) v[j] = __uint_as_float(h[j]) + __uint_as_float(l[j]);
        } else {
#pragma unroll
          for (int c = 0; c + 16 <= CB; c += 16) {
            uint32_t h[16], l[16];
            tc_ld16(taddr + b0 + c, h);
            tc_ld16(taddr + BP + b0 + c, l);
            tc_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) v[c + j] = __uint_as_float(h[j]) + __uint_as_float(l[j]);
          }
        }
        if (whole) {
          if (p.act_mode == ACT_F32_NORM) {
#pragma unroll
            for (int j = 0; j < CB; ++j) v[j] *= rstd_s[b0 + j];
          }
          epi_apply<CB, PUSH>(p, n, b0, v, lane, pos_s, pa, pb, BP, a.wp, push_s);
        } else {
#pragma unroll
          for (int j = 0; j < CB; j += 4) piece[((b0 + j) >> 2) * 32] = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tmem_empty[ab]);
      if (whole) continue;

      // ---- a tile shared with other CTAs: publish the piece; the last arrival adds all pieces in CTA
      // order and finishes the tile
      __threadfence();
      asm volatile("bar.sync 1, 256;" ::: "memory");
      const int c_lo = sp.owner(t * nkb), c_hi = sp.owner((t + 1) * nkb - 1);
      if (et == 0) {
        const int prev = atomicAdd(a.tickets + t, 1);
        const int last = prev == c_hi - c_lo;
        if (last) a.tickets[t] = 0;  // ready for the next launch
        *last_flag = last;
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
      const bool last = *last_flag != 0;
      asm volatile("bar.sync 1, 256;" ::: "memory");  // the flag is rewritten by the next shared tile
      if (!last) continue;
      __threadfence();
      // Up to 16 batch columns at a time with the pieces of up to four CTAs in flight together (16 independent
      // 16-byte loads per thread, issued together with the tail's own reads); every element is still summed in
      // CTA order.
      constexpr int FB = CB;
      const float4* mine = reinterpret_cast<const float4*>(a.partial) + q * (BP / 4) * 32 + lane;
#pragma unroll 1
      for (int b0 = c_begin; b0 < c_end; b0 += FB) {
        float v[FB], pa[FB], pb[FB];
        epi_prefetch<FB>(p, n, b0, lane, pos_s, pa, pb);
#pragma unroll
        for (int j = 0; j < FB; ++j) v[j] = 0.f;
#pragma unroll 1
        for (int c0 = c_lo; c0 <= c_hi; c0 += 4) {
          float4 x[4][FB / 4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int c = min(c0 + u, c_hi);
            const int slot = (t == sp.start(c) / nkb) ? 0 : 1;
            const float4* src = mine + (static_cast<size_t>(c) * 2 + slot) * (BP * BM / 4) + (b0 >> 2) * 32;
#pragma unroll
            for (int g = 0; g < FB / 4; ++g) x[u][g] = __ldcg(src + g * 32);
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            if (c0 + u > c_hi) break;
#pragma unroll
            for (int g = 0; g < FB / 4; ++g) {
              v[4 * g] += x[u][g].x, v[4 * g + 1] += x[u][g].y, v[4 * g + 2] += x[u][g].z, v[4 * g + 3] += x[u][g].w;
            }
          }
        }
        if (p.act_mode == ACT_F32_NORM) {
#pragma unroll
          for (int j = 0; j < FB; ++j) v[j] *= rstd_s[b0 + j];
        }
        epi_apply<FB, PUSH>(p, n, b0, v, lane, pos_s, pa, pb, BP, a.wp, push_s);
      }
    }
    if (!ok && lane == 0 && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "n"(2 * NP < 32 ? 32 : 2 * NP)
                 : "memory");
  }
}

// ---------------------------------------------------------------- host
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn g_encode_wide = nullptr;

cudaError_t make_map(CUtensorMap* map, const void* base, int rows, int K, int box_rows) {
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(K) * 2};
  const cuuint32_t box[2] = {BK, static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = g_encode_wide(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                                   estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

int padded_batch(int batch) { return batch <= 8 ? 8 : (batch <= 16 ? 16 : (batch <= 32 ? 32 : 64)); }

// scratch layout in floats: [64 x kWideMaxSlices] sums of squares | [kWideMaxTiles] tickets | staged activations
// (2 bp x K bf16) | pieces
constexpr int kWideMaxSlices = 64;  // K up to 131072
size_t stage_offset() { return 64 * kWideMaxSlices + kWideMaxTiles; }
size_t piece_offset(int bp, int K) { return stage_offset() + ((static_cast<size_t>(bp) * K + 3) & ~size_t(3)); }

// How many CTAs a launch gets.  The K-block-tiles are cut into equal contiguous ranges, and a tile whose K range is
// cut costs a fix-up at the end of the launch (pieces through L2, a ticket, the last arrival adds them up): about
// 1.5 us at batch <= 8, 3 us at 16, 6 us at 32, 10 us at 64.  When a slightly smaller grid cuts the work at tile boundaries only,
// or cuts every tile into the same whole number of ranges, and the streaming time it gives up (every CTA streams
// about 45 GB/s) is less than that fix-up, it is the better grid - which only ever happens for the short launches
// of small layers (TP-rank slice, ms per step with / without: batch 64 7.82 / 8.22, batch 16 with standard residuals
// 6.35 / 6.55, ladder batch 16 and the 70B shape unchanged).
int pick_grid(int tiles, int nkb, int avail, int bp, double weight_bytes) {
  const int total = tiles * nkb;
  if (total <= avail) return total;
  auto aligned = [&](int g) {
    if (total % g) return false;
    const int per = total / g;
    return per % nkb == 0 || nkb % per == 0;
  };
  if (aligned(avail)) return avail;
  const double fix_us = bp <= 8 ? 1.5 : (bp == 16 ? 3.0 : (bp == 32 ? 6.0 : 10.0));
  const double us_per_cta = weight_bytes / 45e3;  // streaming time if one CTA did it all
  const double t_avail = us_per_cta / avail + fix_us;
  for (int g = avail - 1; g >= 1 && us_per_cta / g < t_avail; --g)
    if (aligned(g)) return g;
  return avail;
}

template <int NP>
cudaError_t launch_np(const WideArgs& a, const CUtensorMap& mw, const CUtensorMap& ma, int grid, cudaStream_t stream,
                      bool pdl_attr) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kWideThreads);
  cfg.dynamicSmemBytes = WCfg<NP>::SMEM;
  cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // the staging kernel, or the producer of a staged operand
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl_attr ? 1 : 0;
  if (a.wp.push_channel) return cudaLaunchKernelEx(&cfg, decode_gemm_wide_tc_kernel<NP, true>, a, mw, ma);
  return cudaLaunchKernelEx(&cfg, decode_gemm_wide_tc_kernel<NP, false>, a, mw, ma);
}

template <int NP>
cudaError_t allow_smem() {
  cudaError_t e = cudaFuncSetAttribute(decode_gemm_wide_tc_kernel<NP, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       WCfg<NP>::SMEM);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(decode_gemm_wide_tc_kernel<NP, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             WCfg<NP>::SMEM);
  return e;
}

}  // namespace


int wide_padded_batch(int batch) { return padded_batch(batch); }

cudaError_t smallm_gemm_wide_tc_init() {
  if (!g_encode_wide) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    g_encode_wide = reinterpret_cast<EncodeFn>(fn);
  }
  cudaError_t e = allow_smem<16>();
  if (e == cudaSuccess) e = allow_smem<32>();
  if (e == cudaSuccess) e = allow_smem<64>();
  if (e == cudaSuccess) e = allow_smem<128>();
  return e;
}

size_t smallm_gemm_wide_tc_scratch_floats(int N, int K, int batch) {
  (void)N;
  const int bp = padded_batch(batch);
  return piece_offset(bp, K) + static_cast<size_t>(kWideMaxCtas) * 2 * bp * BM;
}

size_t smallm_gemm_wide_tc_smem_bytes(int batch) {
  const int bp = padded_batch(batch);
  return bp == 8 ? WCfg<16>::SMEM : (bp == 16 ? WCfg<32>::SMEM : (bp == 32 ? WCfg<64>::SMEM : WCfg<128>::SMEM));
}

namespace {
cudaError_t launch_stage(const SmallMParams& p, int bp, int n_slices, __nv_bfloat16* stage, float* ssq, cudaStream_t stream,
                         bool pdl) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(bp, n_slices);
  cfg.blockDim = dim3(256);
  cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  StagePull pl = {};
  if (p.wide_peer && p.wide_peer->peer.world > 0 && (p.wide_peer->pull_channel[0] | p.wide_peer->pull_channel[1])) {
    const WidePeer& wp = *p.wide_peer;
    if (wp.pull_channel[0] && wp.pull_channel[0] == wp.pull_channel[1]) return cudaErrorInvalidValue;
    pl.peer = wp.peer;
    pl.channel[0] = wp.pull_channel[0];
    pl.channel[1] = wp.pull_channel[1];
    pl.status = p.status;
  }
  return cudaLaunchKernelEx(&cfg, wide_stage_kernel, static_cast<const float*>(p.act), p.gain,
                            p.act_mode == ACT_F32_NORM ? 1 : 0, p.batch, bp, p.K, stage, ssq, p.act_pending,
                            p.act_pending2, p.act_sum_out, pl);
}
}  // namespace

cudaError_t launch_smallm_gemm_wide_stage(const SmallMParams& p, cudaStream_t stream, bool pdl) {
  if (!p.scratch || !p.act || p.batch < 1 || p.batch > 64 || (p.K & 7)) return cudaErrorInvalidValue;
  const int bp = padded_batch(p.batch);
  const int n_slices = (p.K + kStageSlice - 1) / kStageSlice;
  if (n_slices > kWideMaxSlices) return cudaErrorInvalidValue;
  return launch_stage(p, bp, n_slices, reinterpret_cast<__nv_bfloat16*>(p.scratch + stage_offset()), p.scratch, stream, pdl);
}

cudaError_t launch_smallm_gemm_wide_tc(const SmallMParams& p, cudaStream_t stream, bool pdl, int sm_count) {
  if (!g_encode_wide) return cudaErrorNotReady;
  if (!p.scratch || p.batch < 1 || p.batch > 64 || (p.K & 7) || (p.N & 1)) return cudaErrorInvalidValue;
  if ((reinterpret_cast<uintptr_t>(p.W) | reinterpret_cast<uintptr_t>(p.scratch)) & 15) return cudaErrorMisalignedAddress;
  const bool push = p.wide_peer && p.wide_peer->push_channel;
  if (push && ((p.epi_mode != EPI_PLAIN && p.epi_mode != EPI_RESID) || p.wide_peer->peer.world < 1 || p.wide_peer->push_channel > 2 ||
               static_cast<size_t>(p.batch) * p.N > p.wide_peer->peer.max_floats))
    return cudaErrorInvalidValue;
  const int bp = padded_batch(p.batch);
  const int tiles = (p.N + BM - 1) / BM, nkb = (p.K + BK - 1) / BK;
  if (tiles > kWideMaxTiles || sm_count > kWideMaxCtas) return cudaErrorInvalidValue;
  float* ssq = p.scratch;
  int32_t* tickets = reinterpret_cast<int32_t*>(p.scratch + 64 * kWideMaxSlices);
  const int n_slices = (p.K + kStageSlice - 1) / kStageSlice;
  if (n_slices > kWideMaxSlices) return cudaErrorInvalidValue;
  __nv_bfloat16* stage = reinterpret_cast<__nv_bfloat16*>(p.scratch + stage_offset());
  float* pieces = p.scratch + piece_offset(bp, p.K);

  if (p.act_staged) {  // the producing kernel has written the operand already
    if (p.act_mode != ACT_F32 || (reinterpret_cast<uintptr_t>(p.act_staged) & 15)) return cudaErrorInvalidValue;
    stage = const_cast<__nv_bfloat16*>(p.act_staged);
  } else if (!p.wide_prestaged) {  // 1. activations -> bf16 hi + lo, 1/rms
    cudaError_t e = launch_stage(p, bp, n_slices, stage, ssq, stream, pdl);
    if (e != cudaSuccess) return e;
  }
  CUtensorMap mw, ma;
  cudaError_t e = make_map(&mw, p.W, p.N, p.K, BM);
  if (e == cudaSuccess) e = make_map(&ma, stage, 2 * bp, p.K, 2 * bp);
  if (e != cudaSuccess) return e;
  WideArgs a = {};
  a.p = p;
  a.bp = bp;
  a.tiles = tiles;
  a.nkb = nkb;
  a.ssq = ssq;
  a.n_slices = n_slices;
  a.partial = pieces;
  a.tickets = tickets;
  if (push) a.wp = *p.wide_peer;
  a.p.wide_peer = nullptr;  // a host address: not for the device
  const int total = tiles * nkb;
  const int grid = pick_grid(tiles, nkb, sm_count, bp, static_cast<double>(p.N) * p.K * 2.0);
  const bool pdl_attr = (p.act_staged || p.wide_prestaged) ? pdl : true;  // after its own staging kernel always; else if the caller says so
  if (bp == 8) return launch_np<16>(a, mw, ma, grid, stream, pdl_attr);
  if (bp == 16) return launch_np<32>(a, mw, ma, grid, stream, pdl_attr);
  if (bp == 32) return launch_np<64>(a, mw, ma, grid, stream, pdl_attr);
  return launch_np<128>(a, mw, ma, grid, stream, pdl_attr);
}

}  // namespace ladder
