// Large-M GEMM of the prefill path:  C[m, n] = sum_k A[m, k] * W[n, k]   (A bf16 [M,K], W bf16 [N,K], fp32 accumulate)
// with the fused epilogues of the layer: residual add (Eq. 1 / Eq. 2 of the paper), SwiGLU over
// interleaved gate/up rows, rotary embedding + KV-cache append, plain stores.
//
// Activations may come as a bf16 hi + lo pair (a ~ hi + lo): both tiles are staged and multiplied
// with the same weight tile, which removes the activation rounding error at twice the MMA count.
//
// This file holds the dispatcher and the warp-level (mma.sync) implementation, kept as the second
// opinion the tcgen05 kernel (prefill_gemm_tc.cu) is tested against: 128x128x32 CTA tiles, 3-stage
// cp.async pipeline, ldmatrix fragments, 8 warps of 64x32.  Adjacent output columns (2j, 2j+1)
// live in one thread, which is what the pair-wise epilogues (SwiGLU, rotary) need.
#include "common.cuh"
#include "kernels.h"
#include "prefill_epilogue.cuh"

namespace ladder {
namespace {

constexpr int BM = 128, BN = 128, BK = 32, STAGES = 3, PITCH = BK + 8;  // pitch in elements (80 bytes)
constexpr int kGemmThreads = 256;
constexpr int kTileElems = BM * PITCH;
constexpr int kSmemBytes = STAGES * 3 * kTileElems * 2;  // A hi, A lo, W

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;  // zero-fill when out of range
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}

template <bool SPLIT>
__global__ void __launch_bounds__(kGemmThreads) largem_gemm_kernel(const LargeMParams p) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  __nv_bfloat16* sA = reinterpret_cast<__nv_bfloat16*>(smem_raw);
  __nv_bfloat16* sB = sA + STAGES * kTileElems;
  __nv_bfloat16* sL = sB + STAGES * kTileElems;  // lo part of A

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int wm = warp >> 2, wn = warp & 3;  // 2 x 4 warps, warp tile 64 x 32
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int nk = (p.K + BK - 1) / BK;

  // each thread copies 2 x 16 B of A and 2 x 16 B of W per stage: row = (tid>>2) + 64*i, chunk = tid&3
  auto load_stage = [&](int kt, int st) {
    const int kc = kt * BK + (tid & 3) * 8;
    const bool kv = kc < p.K;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int r = (tid >> 2) + 64 * i;
      const int m = m0 + r, n = n0 + r;
      const bool va = kv && m < p.M, vb = kv && n < p.N;
      const __nv_bfloat16* ga = p.A + (va ? static_cast<size_t>(m) * p.K + kc : 0);
      const __nv_bfloat16* gb = p.W + (vb ? static_cast<size_t>(n) * p.K + kc : 0);
      cp_async16(smem_u32(sA + st * kTileElems + r * PITCH + (tid & 3) * 8), ga, va);
      cp_async16(smem_u32(sB + st * kTileElems + r * PITCH + (tid & 3) * 8), gb, vb);
      if (SPLIT) {
        const __nv_bfloat16* gl = p.A_lo + (va ? static_cast<size_t>(m) * p.K + kc : 0);
        cp_async16(smem_u32(sL + st * kTileElems + r * PITCH + (tid & 3) * 8), gl, va);
      }
    }
  };

  float acc[4][4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[i][j][c] = 0.f;

  for (int s = 0; s < STAGES - 1; ++s) {
    if (s < nk) load_stage(s, s);
    cp_async_commit();
  }
  for (int kt = 0; kt < nk; ++kt) {
    cp_async_wait<STAGES - 2>();
    __syncthreads();
    const int nxt = kt + STAGES - 1;
    if (nxt < nk) load_stage(nxt, nxt % STAGES);
    cp_async_commit();
    const __nv_bfloat16* a = sA + (kt % STAGES) * kTileElems;
    const __nv_bfloat16* b = sB + (kt % STAGES) * kTileElems;
    const __nv_bfloat16* al = sL + (kt % STAGES) * kTileElems;
#pragma unroll
    for (int ks = 0; ks < BK; ks += 16) {
      uint32_t af[4][4], bfr[2][4];
#pragma unroll
      for (int j = 0; j < 2; ++j)
        ldmatrix_x4(smem_u32(b + (wn * 32 + j * 16 + (lane & 7) + (lane >> 4) * 8) * PITCH + ks + ((lane >> 3) & 1) * 8),
                    bfr[j][0], bfr[j][1], bfr[j][2], bfr[j][3]);
#pragma unroll
      for (int part = 0; part < (SPLIT ? 2 : 1); ++part) {
        const __nv_bfloat16* src = part ? al : a;
#pragma unroll
        for (int i = 0; i < 4; ++i)
          ldmatrix_x4(smem_u32(src + (wm * 64 + i * 16 + (lane & 15)) * PITCH + ks + (lane >> 4) * 8), af[i][0],
                      af[i][1], af[i][2], af[i][3]);
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j)
            mma_bf16_16816(acc[i][j], af[i][0], af[i][1], af[i][2], af[i][3], bfr[j >> 1][(j & 1) * 2],
                           bfr[j >> 1][(j & 1) * 2 + 1]);
      }
    }
  }
  cp_async_wait<0>();

  const int g = lane >> 2, tig = lane & 3;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int m = m0 + wm * 64 + i * 16 + g;
      const int n = n0 + wn * 32 + j * 8 + tig * 2;
      epilogue_pair(p, m, n, acc[i][j][0], acc[i][j][1]);
      epilogue_pair(p, m + 8, n, acc[i][j][2], acc[i][j][3]);
    }
}

}  // namespace

cudaError_t largem_gemm_init() {
  cudaError_t e = cudaFuncSetAttribute(largem_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(largem_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
}

namespace {
int g_prefill_impl = 0;
int g_sm_count = 0;
}  // namespace

void set_prefill_gemm_impl(int impl) { g_prefill_impl = impl >= 1 && impl <= 3 ? impl : 0; }
bool prefill_single_bf16() { return g_prefill_impl == 2; }
int prefill_gemm_impl() { return g_prefill_impl; }

cudaError_t launch_largem_gemm(const LargeMParams& p, cudaStream_t stream) {
  if (g_prefill_impl != 1 || p.f16) {
    if (!g_sm_count) {
      int dev = 0;
      if (cudaGetDevice(&dev) != cudaSuccess ||
          cudaDeviceGetAttribute(&g_sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        g_sm_count = 148;
    }
    return launch_largem_gemm_tc(p, stream, g_sm_count);
  }
  dim3 grid((p.N + BN - 1) / BN, (p.M + BM - 1) / BM);
  if (p.A_lo) largem_gemm_kernel<true><<<grid, kGemmThreads, kSmemBytes, stream>>>(p);
  else largem_gemm_kernel<false><<<grid, kGemmThreads, kSmemBytes, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace ladder
