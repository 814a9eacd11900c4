// Weight-streaming small-M GEMM for the decode path:  acc[b, n] = sum_k act[b, k] * W[n, k],  b < batch <= 64.
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
//   * activations are staged per K-chunk by the consumer warps (fp32 residual x gain -> bf16,
//     sum of squares accumulated on the way, so RMSNorm costs one pass and its 1/rms factor is
//     applied to the accumulators in the epilogue);
//   * everything that does not depend on the previous kernel (barrier set-up, the first ring
//     fill of weights) happens before griddepcontrol.wait, so with programmatic dependent
//     launch the weight stream never drains between kernels;
//   * epilogues: residual add (Eq. 1 / Eq. 2 of the paper: destination = addend + h), SwiGLU
//     over interleaved gate/up rows, rotary embedding + KV-cache append, plain store.
// Results are deterministic: the K split across warps is reduced in a fixed order.
#include "common.cuh"
#include "kernels.h"

namespace ladder {
namespace {

constexpr int kThreads = 160;  // warp 0 = producer, warps 1..4 = consumers

template <int NB>
struct Cfg {
  static constexpr int TK = NB == 1 ? 1024 : (NB == 2 ? 512 : 256);  // K elements per chunk
  static constexpr int STAGES = NB == 1 ? 4 : (NB == 2 ? 8 : 12);
  static constexpr int PITCH = TK * 2 + 64;  // bytes between weight rows in a stage (64 mod 128)
  static constexpr int STAGE_BYTES = 16 * PITCH;
  static constexpr int APITCH = TK * 2 + 64;
  static constexpr int ACT_ROWS = 8 * NB;
  static constexpr int ACT_BYTES = ACT_ROWS * APITCH;
  static constexpr int RG_MAX = 8 / NB;    // 16-row groups whose accumulators live in registers at once
  static constexpr int SPW = TK / 32 / 4;  // 32-wide K slabs per consumer warp per chunk
  static constexpr int KQ = TK / 8;        // 16-byte units per activation row per chunk
  static constexpr int RL = 128 / KQ;      // consumer threads side by side along the batch
  static constexpr int RPT = ACT_ROWS / RL;  // activation rows per thread
  static constexpr int PF = RPT < 4 ? RPT : 4;  // rows prefetched into registers one chunk ahead
  static constexpr int RED_FLOATS = 4 * RG_MAX * NB * 4 * 32;
  static constexpr int SMEM = STAGES * STAGE_BYTES + 2 * ACT_BYTES + RED_FLOATS * 4 + (4 * 16 + 64) * 4 +
                              2 * STAGES * 8 + 16 + 128;
};

struct F8 {
  float4 a, b;
};

template <int NB, int ACT>
__global__ void __launch_bounds__(kThreads, 1) smallm_gemm_kernel(const SmallMParams p) {
  using C = Cfg<NB>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  uint8_t* ring = smem;
  uint8_t* act = ring + C::STAGES * C::STAGE_BYTES;
  float* red = reinterpret_cast<float*>(act + 2 * C::ACT_BYTES);
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

    // register prefetch of the raw activation chunk
    F8 pf_x[C::PF];
    uint4 pf_h[C::PF];
    uint4 pf_g = make_uint4(0, 0, 0, 0);
    auto prefetch = [&](int ch) {
      const int k = ch * C::TK + kq * 8;
      const bool kv = k < p.K;
      if (ACT == ACT_F32_NORM) {
        pf_g = kv ? __ldg(reinterpret_cast<const uint4*>(p.gain + k)) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int i = 0; i < C::PF; ++i) {
          const int b = rl + i * C::RL;
          if (kv && b < batch) {
            const float4* src = reinterpret_cast<const float4*>(static_cast<const float*>(p.act) +
                                                                static_cast<size_t>(b) * p.K + k);
            pf_x[i].a = src[0];
            pf_x[i].b = src[1];
          } else {
            pf_x[i].a = make_float4(0, 0, 0, 0);
            pf_x[i].b = make_float4(0, 0, 0, 0);
          }
        }
      } else {
#pragma unroll
        for (int i = 0; i < C::PF; ++i) {
          const int b = rl + i * C::RL;
          pf_h[i] = (kv && b < batch)
                        ? *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(p.act) +
                                                          static_cast<size_t>(b) * p.K + k)
                        : make_uint4(0, 0, 0, 0);
        }
      }
    };
    auto norm_pack = [&](const F8& x, const uint4& gq, float& ss) -> uint4 {
      ss += x.a.x * x.a.x + x.a.y * x.a.y + x.a.z * x.a.z + x.a.w * x.a.w + x.b.x * x.b.x + x.b.y * x.b.y +
            x.b.z * x.b.z + x.b.w * x.b.w;
      uint4 o;
      o.x = pack_bf16x2(x.a.x * bf16_lo(gq.x), x.a.y * bf16_hi(gq.x));
      o.y = pack_bf16x2(x.a.z * bf16_lo(gq.y), x.a.w * bf16_hi(gq.y));
      o.z = pack_bf16x2(x.b.x * bf16_lo(gq.z), x.b.y * bf16_hi(gq.z));
      o.w = pack_bf16x2(x.b.z * bf16_lo(gq.w), x.b.w * bf16_hi(gq.w));
      return o;
    };
    auto stage_act = [&](int ch) {
      const uint32_t dst = act_u32 + (ch & 1) * C::ACT_BYTES + kq * 16;
      const int k = ch * C::TK + kq * 8;
      const bool kv = k < p.K;
#pragma unroll
      for (int i = 0; i < C::RPT; ++i) {
        const int b = rl + i * C::RL;
        if (b >= batch) break;
        uint4 o;
        if (i < C::PF) {
          if (ACT == ACT_F32_NORM) o = norm_pack(pf_x[i < C::PF ? i : 0], pf_g, ssq[i]);
          else o = pf_h[i < C::PF ? i : 0];
        } else {
          if (ACT == ACT_F32_NORM) {
            F8 x;
            x.a = x.b = make_float4(0, 0, 0, 0);
            if (kv) {
              const float4* src = reinterpret_cast<const float4*>(static_cast<const float*>(p.act) +
                                                                  static_cast<size_t>(b) * p.K + k);
              x.a = src[0];
              x.b = src[1];
            }
            o = norm_pack(x, pf_g, ssq[i]);
          } else {
            o = kv ? *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(p.act) +
                                                     static_cast<size_t>(b) * p.K + k)
                   : make_uint4(0, 0, 0, 0);
          }
        }
        sts128(dst + b * C::APITCH, o);
      }
    };

    prefetch(0);
    for (int ch = 0; ch < nchunk; ++ch) {
      stage_act(ch);
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (ch + 1 < nchunk) prefetch(ch + 1);

      // activation fragments of this warp's K slabs (reused by every row group of the pass)
      uint4 bf[C::SPW][NB];
      const int k0 = ch * C::TK;
#pragma unroll
      for (int j = 0; j < C::SPW; ++j)
#pragma unroll
        for (int nt = 0; nt < NB; ++nt) {
          const int brow = nt * 8 + g;
          bf[j][nt] = brow < batch ? lds128(act_u32 + (ch & 1) * C::ACT_BYTES + brow * C::APITCH +
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
          for (int nt = 0; nt < NB; ++nt) {
            mma_bf16_16816(acc[rgi][nt], lo.x, hi.x, lo.y, hi.y, bf[j][nt].x, bf[j][nt].y);
            mma_bf16_16816(acc[rgi][nt], lo.z, hi.z, lo.w, hi.w, bf[j][nt].z, bf[j][nt].w);
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
    if (ACT == ACT_F32_NORM) {
#pragma unroll
      for (int i = 0; i < C::RPT; ++i) {
        const float s = warp_sum(ssq[i]);
        if (lane == 0) ssq_s[cw * 16 + i] = s;
      }
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (ACT == ACT_F32_NORM) {
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
      if (ACT == ACT_F32_NORM) s *= rstd_s[b];
      return s;
    };

    if (p.epi_mode == EPI_RESID || p.epi_mode == EPI_PLAIN) {
      float* out = static_cast<float*>(p.out);
      for (int idx = ct; idx < prow * batch; idx += 128) {
        const int r = idx % prow, b = idx / prow;
        const size_t o = static_cast<size_t>(b) * p.N + nbase + r;
        float v = value(r, b);
        if (p.epi_mode == EPI_RESID) v += p.addend[o];
        out[o] = v;
      }
    } else if (p.epi_mode == EPI_SWIGLU) {
      __nv_bfloat16* out = static_cast<__nv_bfloat16*>(p.out);
      const int half = prow >> 1;
      for (int idx = ct; idx < half * batch; idx += 128) {
        const int pr = idx % half, b = idx / half;
        const float gt = value(2 * pr, b), up = value(2 * pr + 1, b);
        const float h = gt / (1.f + __expf(-gt)) * up;
        out[static_cast<size_t>(b) * (p.N >> 1) + ((nbase >> 1) + pr)] = __float2bfloat16_rn(h);
      }
    } else if (p.epi_mode == EPI_QKV_ROPE) {
      const QkvEpilogue& e = p.qkv;
      const int half = prow >> 1, Dh = e.head_dim;
      const int nq = e.n_q_heads * Dh, nk = e.n_kv_heads * Dh;
      for (int idx = ct; idx < half * batch; idx += 128) {
        const int pr = idx % half, b = idx / half;
        const int n = nbase + 2 * pr;
        float v0 = value(2 * pr, b), v1 = value(2 * pr + 1, b);
        const int pos = e.seq_lens[b];
        if (pos < 0 || pos >= e.max_seq_len) {
          if (p.status) atomicOr(p.status, LADDER_DEV_CACHE_OVERFLOW);
          continue;
        }
        if (n < nq + nk) {  // rotate q and k pairs
          const float2 cs = e.rope[static_cast<size_t>(pos) * (Dh >> 1) + ((n % Dh) >> 1)];
          const float a0 = v0 * cs.x - v1 * cs.y, a1 = v0 * cs.y + v1 * cs.x;
          v0 = a0;
          v1 = a1;
        }
        if (n < nq) {
          *reinterpret_cast<float2*>(e.q_out_f32 + static_cast<size_t>(b) * nq + n) = make_float2(v0, v1);
        } else {
          const int nn = n < nq + nk ? n - nq : n - nq - nk;
          __nv_bfloat16* cache = n < nq + nk ? e.k_cache : e.v_cache;
          const size_t off =
              ((static_cast<size_t>(b) * e.n_kv_heads + nn / Dh) * e.max_seq_len + pos) * Dh + (nn % Dh);
          *reinterpret_cast<uint32_t*>(cache + off) = pack_bf16x2(v0, v1);
        }
      }
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");  // red / rstd are reused by the next pass
  }
  if (!ok && lane == 0 && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
}

template <int NB>
cudaError_t launch_nb(const SmallMParams& p, cudaStream_t stream, bool pdl, int grid) {
  using C = Cfg<NB>;
  auto kern = p.act_mode == ACT_F32_NORM ? smallm_gemm_kernel<NB, ACT_F32_NORM> : smallm_gemm_kernel<NB, ACT_BF16>;
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

template <int NB>
cudaError_t init_nb() {
  cudaError_t e = cudaFuncSetAttribute(smallm_gemm_kernel<NB, ACT_F32_NORM>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<NB>::SMEM);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(smallm_gemm_kernel<NB, ACT_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              Cfg<NB>::SMEM);
}

}  // namespace

cudaError_t smallm_gemm_init() {
  cudaError_t e = init_nb<1>();
  if (e == cudaSuccess) e = init_nb<2>();
  if (e == cudaSuccess) e = init_nb<4>();
  if (e == cudaSuccess) e = init_nb<8>();
  return e;
}

size_t smallm_gemm_smem_bytes(int batch) {
  if (batch <= 8) return Cfg<1>::SMEM;
  if (batch <= 16) return Cfg<2>::SMEM;
  if (batch <= 32) return Cfg<4>::SMEM;
  return Cfg<8>::SMEM;
}

cudaError_t launch_smallm_gemm(const SmallMParams& p, cudaStream_t stream, bool pdl, int sm_count) {
  const int units = p.N >> 3;
  const int grid = units < sm_count ? units : sm_count;
  if (p.batch <= 8) return launch_nb<1>(p, stream, pdl, grid);
  if (p.batch <= 16) return launch_nb<2>(p, stream, pdl, grid);
  if (p.batch <= 32) return launch_nb<4>(p, stream, pdl, grid);
  return launch_nb<8>(p, stream, pdl, grid);
}

}  // namespace ladder
