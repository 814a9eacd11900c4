// Weight-streaming small-M GEMM for the decode path, batches 9..64 (batch <= 8 has its own kernel
// in decode_gemm.cu):  acc[b, n] = sum_k act[b, k] * W[n, k].
//
// The kernel is HBM-bound: every weight byte is read exactly once and nothing else of size
// is touched.  Design:
//   * persistent grid of one CTA per SM; CTA c owns a contiguous range of 8-row units of W
//     (contiguous in memory because W is row-major with K contiguous);
//   * one producer warp streams [16 rows x TK] weight tiles into a shared-memory ring with 1-D
//     bulk async copies (TMA engine) signalling mbarriers, L2 evict-first;
//   * four consumer warps split each tile along K and feed mma.sync m16n8k16 (weights = A
//     operand, activations = B operand, batch padded to 8*NB columns).  Each thread reads 16
//     contiguous bytes of a weight row and the matching 16 bytes of an activation row: the K
//     index inside an MMA is permuted the same way for both operands, so no ldmatrix and no
//     swizzle are needed; a row pitch of 64 mod 128 bytes keeps the 128-bit loads conflict-free;
//   * activations are fp32 in global memory and are staged per K-chunk by the consumer warps:
//     (x * gain) is split into a bf16 high part and a bf16 low part (x ~ hi + lo, ~16 mantissa
//     bits) and both are multiplied with the weight fragment, so the tensor-core operands are
//     bf16 while the activation rounding error all but disappears -- the extra MMAs are free in
//     a bandwidth-bound kernel.  The sum of squares is accumulated on the way, so RMSNorm costs
//     one pass and its 1/rms factor is applied to the accumulators in the epilogue;
//   * everything that does not depend on the previous kernel (barrier set-up, the first ring
//     fill of weights) happens before griddepcontrol.wait, so with programmatic dependent
//     launch the weight stream never drains between kernels;
//   * epilogues: residual add (Eq. 1 / Eq. 2 of the paper: destination = addend + h), SwiGLU
//     over interleaved gate/up rows, rotary embedding + KV-cache append, plain store.
// Results are deterministic: the K split across warps is reduced in a fixed order.
#include "common.cuh"
#include "kernels.h"
#include "smallm_epilogue.cuh"

namespace ladder {
namespace {

constexpr int kThreads = 160;  // warp 0 = producer, warps 1..4 = consumers

template <int NB, bool R4>
struct Cfg {
  static constexpr int TK = NB == 1 ? 1024 : (NB == 2 ? 512 : 256);  // K elements per chunk
  static constexpr int STAGES = NB == 1 ? 4 : (NB == 2 ? 7 : 12);
  static constexpr int PITCH = TK * 2 + 64;  // bytes between weight rows in a stage (64 mod 128)
  static constexpr int STAGE_BYTES = 16 * PITCH;
  static constexpr int APITCH = TK * 2 + 64;
  static constexpr bool SPLIT = NB <= 2;     // activations as bf16 hi + lo pair (batch <= 16)
  static constexpr int PARTS = SPLIT ? 2 : 1;
  static constexpr int ACT_ROWS = R4 ? 4 : 8 * NB;  // R4: batch <= 4 needs only 4 staged rows
  static constexpr int ACT_BYTES = ACT_ROWS * APITCH;
  static constexpr int RG_MAX = 8 / NB;    // 16-row groups whose accumulators live in registers at once
  static constexpr int SPW = TK / 32 / 4;  // 32-wide K slabs per consumer warp per chunk
  static constexpr int KQ = TK / 8;        // 16-byte units per activation row per chunk
  static constexpr int RL = 128 / KQ;      // consumer threads side by side along the batch
  static constexpr int RPT = (ACT_ROWS + RL - 1) / RL;  // activation rows per thread
  static constexpr int PF = RPT < 4 ? RPT : 4;  // rows prefetched into registers one chunk ahead
  static constexpr int RED_FLOATS = 4 * RG_MAX * NB * 4 * 32;
  static constexpr int SMEM = STAGES * STAGE_BYTES + 2 * PARTS * ACT_BYTES + RED_FLOATS * 4 + (4 * 16 + 64) * 4 +
                              2 * STAGES * 8 + 16 + 128;
  static_assert(!R4 || NB == 1, "R4 is a variant of the batch <= 8 kernel");
  static_assert(SMEM <= 232448, "exceeds the 227 KB of shared memory a CTA can opt in to");
};

struct F8 {
  float4 a, b;
};

template <int NB, bool R4, bool NORM>
__global__ void __launch_bounds__(kThreads, 1) smallm_gemm_kernel(const SmallMParams p) {
  using C = Cfg<NB, R4>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  uint8_t* ring = smem;
  uint8_t* act = ring + C::STAGES * C::STAGE_BYTES;
  float* red = reinterpret_cast<float*>(act + 2 * C::PARTS * C::ACT_BYTES);
  float* ssq_s = red + C::RED_FLOATS;  // [4 warps][16]
  float* rstd_s = ssq_s + 64;          // [64]
  uint64_t* full = reinterpret_cast<uint64_t*>(rstd_s + 64);
  uint64_t* empty = full + C::STAGES;
  int* flag_s = reinterpret_cast<int*>(empty + C::STAGES);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // work partition: contiguous ranges of 8-row units
  const int U = p.N >> 3;
  const int G = gridDim.x;
  const int u0 = static_cast<int>(static_cast<long long>(U) * blockIdx.x / G);
  const int u1 = static_cast<int>(static_cast<long long>(U) * (blockIdx.x + 1) / G);
  const int r0 = u0 * 8, nrows = (u1 - u0) * 8;
  const int nrg = (nrows + 15) >> 4;
  const int npass = (nrg + C::RG_MAX - 1) / C::RG_MAX;
  const int nchunk = (p.K + C::TK - 1) / C::TK;

  if (tid == 0) {
    int dead = 0;
    if (p.status) dead = (*reinterpret_cast<volatile int32_t*>(p.status) & LADDER_DEV_TIMEOUT) ? 1 : 0;
    *flag_s = dead;
    for (int s = 0; s < C::STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 4);
    }
    fence_barrier_init();
  }
  __syncthreads();
  pdl_launch_dependents();
  if (*flag_s || nrows == 0) return;  // an earlier kernel reported a protocol error: do nothing

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    const uint64_t pol = l2_policy_evict_first();
    const uint8_t* Wb = reinterpret_cast<const uint8_t*>(p.W);
    bool ok = true;
    int it = 0;
    for (int ps = 0; ps < npass && ok; ++ps) {
      const int rg0 = ps * C::RG_MAX;
      const int rgn = min(C::RG_MAX, nrg - rg0);
      for (int ch = 0; ch < nchunk && ok; ++ch) {
        const int k0 = ch * C::TK;
        const uint32_t kb = static_cast<uint32_t>(min(C::TK, p.K - k0)) * 2u;
        for (int rg = rg0; rg < rg0 + rgn; ++rg, ++it) {
          const int st = it % C::STAGES;
          const uint32_t ph = (it / C::STAGES) & 1;
          ok = mbar_wait_bounded(&empty[st], ph ^ 1u);
          if (!ok) break;
          const int rows_valid = min(16, nrows - rg * 16);
          if (lane == 0) mbar_expect_tx(&full[st], rows_valid * kb);
          __syncwarp();
          if (lane < rows_valid) {
            const size_t row = static_cast<size_t>(r0 + rg * 16 + lane);
            bulk_g2s(ring + st * C::STAGE_BYTES + lane * C::PITCH, Wb + (row * p.K + k0) * 2, kb, &full[st], pol);
          }
        }
      }
    }
    if (!ok) {
      // protocol error: record it, then wait (bounded) for the copies still in flight
      if (lane == 0 && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
      for (int j = 1; j <= C::STAGES && j <= it; ++j) {
        const int i2 = it - j;
        mbar_wait_bounded(&full[i2 % C::STAGES], (i2 / C::STAGES) & 1);
      }
    }
    return;
  }

  // -------------------------------------------------------------------- consumers
  const int ct = tid - 32;       // 0..127
  const int cw = warp - 1;       // 0..3
  const int g = lane >> 2, tig = lane & 3;
  const int rl = ct / C::KQ, kq = ct % C::KQ;
  const int batch = p.batch;
  const uint32_t ring_u32 = smem_u32(ring);
  const uint32_t act_u32 = smem_u32(act);
  bool ok = true;

  pdl_wait();  // activations (and the addend) come from the previous kernel

  int it = 0;
  for (int ps = 0; ps < npass; ++ps) {
    const int rg0 = ps * C::RG_MAX;
    const int rgn = min(C::RG_MAX, nrg - rg0);
    float acc[C::RG_MAX][NB][4];
#pragma unroll
    for (int a = 0; a < C::RG_MAX; ++a)
#pragma unroll
      for (int b = 0; b < NB; ++b)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[a][b][c] = 0.f;
    float ssq[C::RPT];
#pragma unroll
    for (int i = 0; i < C::RPT; ++i) ssq[i] = 0.f;

    // register prefetch of the raw fp32 activation chunk
    F8 pf_x[C::PF];
    uint4 pf_g = make_uint4(0x3f803f80u, 0x3f803f80u, 0x3f803f80u, 0x3f803f80u);  // gain 1.0
    const float* actf = static_cast<const float*>(p.act);
    auto load_x = [&](int b, int k, bool kv) -> F8 {
      F8 x;
      x.a = x.b = make_float4(0, 0, 0, 0);
      if (kv && b < batch) {
        const float4* src = reinterpret_cast<const float4*>(actf + static_cast<size_t>(b) * p.K + k);
        x.a = src[0];
        x.b = src[1];
      }
      return x;
    };
    auto prefetch = [&](int ch) {
      const int k = ch * C::TK + kq * 8;
      const bool kv = k < p.K;
      if (NORM) pf_g = kv ? __ldg(reinterpret_cast<const uint4*>(p.gain + k)) : make_uint4(0, 0, 0, 0);
#pragma unroll
      for (int i = 0; i < C::PF; ++i) pf_x[i] = load_x(rl + i * C::RL, k, kv);
    };
    // y = x * gain, written as bf16 hi (and lo = bf16(y - hi)); sum of squares of x on the way
    auto stage_row = [&](const F8& x, const uint4& gq, float& ss, uint32_t dst) {
      float y[8] = {x.a.x, x.a.y, x.a.z, x.a.w, x.b.x, x.b.y, x.b.z, x.b.w};
      if (NORM) {
        ss += y[0] * y[0] + y[1] * y[1] + y[2] * y[2] + y[3] * y[3] + y[4] * y[4] + y[5] * y[5] + y[6] * y[6] +
              y[7] * y[7];
        y[0] *= bf16_lo(gq.x);
        y[1] *= bf16_hi(gq.x);
        y[2] *= bf16_lo(gq.y);
        y[3] *= bf16_hi(gq.y);
        y[4] *= bf16_lo(gq.z);
        y[5] *= bf16_hi(gq.z);
        y[6] *= bf16_lo(gq.w);
        y[7] *= bf16_hi(gq.w);
      }
      uint4 hi;
      hi.x = pack_bf16x2(y[0], y[1]);
      hi.y = pack_bf16x2(y[2], y[3]);
      hi.z = pack_bf16x2(y[4], y[5]);
      hi.w = pack_bf16x2(y[6], y[7]);
      sts128(dst, hi);
      if (C::SPLIT) {
        uint4 lo;
        lo.x = pack_bf16x2(y[0] - bf16_lo(hi.x), y[1] - bf16_hi(hi.x));
        lo.y = pack_bf16x2(y[2] - bf16_lo(hi.y), y[3] - bf16_hi(hi.y));
        lo.z = pack_bf16x2(y[4] - bf16_lo(hi.z), y[5] - bf16_hi(hi.z));
        lo.w = pack_bf16x2(y[6] - bf16_lo(hi.w), y[7] - bf16_hi(hi.w));
        sts128(dst + C::ACT_BYTES, lo);
      }
    };
    auto stage_act = [&](int ch) {
      const uint32_t dst = act_u32 + (ch & 1) * C::PARTS * C::ACT_BYTES + kq * 16;
      const int k = ch * C::TK + kq * 8;
      const bool kv = k < p.K;
#pragma unroll
      for (int i = 0; i < C::RPT; ++i) {
        const int b = rl + i * C::RL;
        if (b >= batch || b >= C::ACT_ROWS) break;
        if (i < C::PF) stage_row(pf_x[i < C::PF ? i : 0], pf_g, ssq[i], dst + b * C::APITCH);
        else stage_row(load_x(b, k, kv), pf_g, ssq[i], dst + b * C::APITCH);
      }
    };

    prefetch(0);
    for (int ch = 0; ch < nchunk; ++ch) {
      stage_act(ch);
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (ch + 1 < nchunk) prefetch(ch + 1);

      // activation fragments of this warp's K slabs (reused by every row group of the pass)
      uint4 bf[C::PARTS][C::SPW][NB];
      const int k0 = ch * C::TK;
#pragma unroll
      for (int pt = 0; pt < C::PARTS; ++pt)
#pragma unroll
        for (int j = 0; j < C::SPW; ++j)
#pragma unroll
          for (int nt = 0; nt < NB; ++nt) {
            const int brow = nt * 8 + g;
            bf[pt][j][nt] = (brow < batch && brow < C::ACT_ROWS)
                                ? lds128(act_u32 + ((ch & 1) * C::PARTS + pt) * C::ACT_BYTES + brow * C::APITCH +
                                         (cw * C::SPW + j) * 64 + tig * 16)
                                : make_uint4(0, 0, 0, 0);
          }

#pragma unroll
      for (int rgi = 0; rgi < C::RG_MAX; ++rgi) {
        if (rgi >= rgn) break;  // uniform across the CTA
        const int st = it % C::STAGES;
        const uint32_t ph = (it / C::STAGES) & 1;
        if (ok) ok = mbar_wait_bounded(&full[st], ph);
        const uint32_t base = ring_u32 + st * C::STAGE_BYTES + g * C::PITCH + tig * 16;
#pragma unroll
        for (int j = 0; j < C::SPW; ++j) {
          const int slab = cw * C::SPW + j;
          const bool kv = (k0 + slab * 32 + tig * 8) < p.K;
          uint4 lo = make_uint4(0, 0, 0, 0), hi = make_uint4(0, 0, 0, 0);
          if (kv) {
            lo = lds128(base + slab * 64);
            hi = lds128(base + 8 * C::PITCH + slab * 64);
          }
#pragma unroll
          for (int nt = 0; nt < NB; ++nt)
#pragma unroll
            for (int pt = 0; pt < C::PARTS; ++pt) {
              mma_bf16_16816(acc[rgi][nt], lo.x, hi.x, lo.y, hi.y, bf[pt][j][nt].x, bf[pt][j][nt].y);
              mma_bf16_16816(acc[rgi][nt], lo.z, hi.z, lo.w, hi.w, bf[pt][j][nt].z, bf[pt][j][nt].w);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[st]);
        ++it;
      }
    }

    // ---------------------------------------------------------------- pass epilogue
#pragma unroll
    for (int a = 0; a < C::RG_MAX; ++a)
#pragma unroll
      for (int nt = 0; nt < NB; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c) red[(((cw * C::RG_MAX + a) * NB + nt) * 4 + c) * 32 + lane] = acc[a][nt][c];
    if (NORM) {
#pragma unroll
      for (int i = 0; i < C::RPT; ++i) {
        const float s = warp_sum(ssq[i]);
        if (lane == 0) ssq_s[cw * 16 + i] = s;
      }
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (NORM) {
      if (ct < batch) {
        // row b = rl' + i*RL is staged by the warps whose threads have rl == rl'
        const int rlb = ct % C::RL, i = ct / C::RL;
        constexpr int WPR = 4 / C::RL;  // warps per row lane
        float s = 0.f;
        for (int w = 0; w < WPR; ++w) s += ssq_s[(rlb * WPR + w) * 16 + i];
        rstd_s[ct] = rsqrtf(s / static_cast<float>(p.K) + p.eps);
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
    }

    const int prow = min(rgn * 16, nrows - rg0 * 16);
    const int nbase = r0 + rg0 * 16;
    auto value = [&](int r, int b) -> float {
      const int a = r >> 4, rr = r & 15;
      const int idx = (((a * NB + (b >> 3)) * 4) + ((rr >> 3) * 2 + (b & 1))) * 32 + ((rr & 7) * 4 + ((b & 7) >> 1));
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < 4; ++w) s += red[w * (C::RG_MAX * NB * 128) + idx];
      if (NORM) s *= rstd_s[b];
      return s;
    };

    smallm_epilogue(p, ct, prow, nbase, batch, value);
    asm volatile("bar.sync 1, 128;" ::: "memory");  // red / rstd are reused by the next pass
  }
  if (!ok && lane == 0 && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
}

template <int NB, bool R4>
cudaError_t launch_nb(const SmallMParams& p, cudaStream_t stream, bool pdl, int grid) {
  using C = Cfg<NB, R4>;
  auto kern = p.act_mode == ACT_F32_NORM ? smallm_gemm_kernel<NB, R4, true> : smallm_gemm_kernel<NB, R4, false>;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = C::SMEM;
  cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, p);
}

template <int NB, bool R4>
cudaError_t init_nb() {
  cudaError_t e = cudaFuncSetAttribute(smallm_gemm_kernel<NB, R4, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       Cfg<NB, R4>::SMEM);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(smallm_gemm_kernel<NB, R4, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              Cfg<NB, R4>::SMEM);
}

}  // namespace

cudaError_t smallm_gemm_wide_init() {
  cudaError_t e = init_nb<2, false>();
  if (e == cudaSuccess) e = init_nb<4, false>();
  if (e == cudaSuccess) e = init_nb<8, false>();
  return e;
}

size_t smallm_gemm_wide_smem_bytes(int batch) {
  if (batch <= 16) return Cfg<2, false>::SMEM;
  if (batch <= 32) return Cfg<4, false>::SMEM;
  return Cfg<8, false>::SMEM;
}

// batch 9..64
cudaError_t launch_smallm_gemm_wide(const SmallMParams& p, cudaStream_t stream, bool pdl, int sm_count) {
  const int units = p.N >> 3;
  const int grid = units < sm_count ? units : sm_count;
  if (p.batch <= 16) return launch_nb<2, false>(p, stream, pdl, grid);
  if (p.batch <= 32) return launch_nb<4, false>(p, stream, pdl, grid);
  return launch_nb<8, false>(p, stream, pdl, grid);
}

}  // namespace ladder
