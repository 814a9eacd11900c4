// Large-M GEMM of the prefill path on the 5th-generation tensor cores (tcgen05 / UMMA, sm_100a):
//   C[m, n] = sum_k (A_hi[m, k] + A_lo[m, k]) * W[n, k]      A bf16 [M, K] (hi + optional lo), W bf16 [N, K]
// with fp32 accumulators in tensor memory and the fused layer epilogues (residual add of Eq. 1 /
// Eq. 2 of the paper, SwiGLU, rotary + KV-cache append, plain stores).
//
// Persistent CTAs, one per SM, 192 threads in three roles that meet only at mbarriers:
//   warp 0     TMA producer: per 64-wide K block one 128x64 box of A_hi, one of A_lo and one 256x64
//              (or 128x64: see TcCfg) box of W (cp.async.bulk.tensor.2d, 128-byte swizzle, out-of-range
//              rows/columns zero-filled by the TMA unit) into a 3- or 4-stage shared-memory ring;
//   warp 1     MMA issuer: one elected thread issues tcgen05.mma (M 128, N 256, K 16, kind::f16,
//              bf16 x bf16 -> fp32) straight from shared-memory descriptors -- 4 K-steps for the high
//              part and 4 for the low part of A against the same W tile -- and releases ring stages /
//              publishes accumulators with tcgen05.commit.  Owns the TMEM allocation (512 columns =
//              two 128x256 fp32 accumulators, so the epilogue of tile i overlaps the MMAs of tile i+1);
//   warps 2-5  epilogue: each warp reads its 32-lane quarter of the accumulator with tcgen05.ld
//              (32 columns at a time; a thread owns one output row, so the column pairs the SwiGLU and
//              rotary epilogues need are adjacent registers) and writes the result.
// Tiles are visited in bands of 16 M-tiles, M-fastest inside a band, so that the CTAs running at the
// same time work on ~16 x 9 tiles whose A band and W tiles together fit the L2.
// Every wait is bounded; on a protocol error the kernel records it, drains and frees its TMEM.
#include <cuda.h>

#include "common.cuh"
#include "kernels.h"
#include "prefill_epilogue.cuh"

namespace ladder {
namespace {

constexpr int BM = 128, BK = 64, UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2;  // 16 KB
constexpr int kTcThreads = 192;
// Tile width BN = 256 by default; 128 when that leaves SMs without a tile (small M x N: a short prompt, a chunk of a
// prompt, a narrow projection), which doubles the number of tiles at the same bytes per flop for A.
// SPLIT: A comes as a hi + lo pair (two boxes per stage, two MMA rounds per K block); without it a stage is one A box
// and one W box, which leaves room for one more stage.
template <int BN, bool SPLIT>
struct TcCfg {
  static constexpr int B_BYTES = BN * BK * 2;                              // 32 / 16 KB
  static constexpr int W_OFF = (SPLIT ? 2 : 1) * A_BYTES;                  // the W box follows the A box(es)
  static constexpr int STAGE_BYTES = W_OFF + B_BYTES;                      // SPLIT: 64 / 48 KB, else 48 / 32 KB
  static constexpr int STAGES = SPLIT ? (BN == 256 ? 3 : 4) : (BN == 256 ? 4 : 6);
  static constexpr int OFF_BARS = STAGES * STAGE_BYTES;  // full[], empty[], tmem_full[2], tmem_empty[2], tmem slot
  static constexpr int SMEM = OFF_BARS + 24 * 8 + 1024;
  // Instruction descriptor, kind::f16: D fp32 (bit 4), A format bits 7-9 and B format bits 10-12 (0 = binary16,
  // 1 = bf16; always the same for both operands here), both K-major, N >> 3 at bit 17, M >> 4 at bit 24.
  static constexpr uint32_t IDESC_F16 = (1u << 4) | (static_cast<uint32_t>(BN >> 3) << 17) |
                                        (static_cast<uint32_t>(BM >> 4) << 24);
  static constexpr uint32_t IDESC_BF16 = IDESC_F16 | (1u << 7) | (1u << 10);
};
constexpr int GROUP_M = 16;  // M-tiles per rasterisation band

// tile index -> (m tile, n tile): bands of GROUP_M m-tiles, m fastest inside a band
__device__ __forceinline__ void tile_coords(int t, int tiles_m, int tiles_n, int& tm, int& tn) {
  const int per_band = GROUP_M * tiles_n;
  const int band = t / per_band, r = t - band * per_band;
  const int m_first = band * GROUP_M;
  const int band_m = min(GROUP_M, tiles_m - m_first);
  tm = m_first + r % band_m;
  tn = r / band_m;
}

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
          smem_u32(dst)),
      "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// D(tmem) (+)= A(smem desc) * B(smem desc)
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, "
      "%24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor: K-major operand tile of rows x 64 bf16, 128-byte swizzle
// (rows of 128 bytes, 8-row swizzle atoms of 1024 bytes), tile base 1024-byte aligned.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr & 0x3FFFFu) >> 4);  // start address / 16
  d |= static_cast<uint64_t>(1) << 16;                 // leading byte offset (unused for swizzled K-major)
  d |= static_cast<uint64_t>(1024 >> 4) << 32;         // stride byte offset: next 8-row group
  d |= static_cast<uint64_t>(1) << 46;                 // descriptor version (sm_100)
  d |= static_cast<uint64_t>(2) << 61;                 // SWIZZLE_128B
  return d;
}

template <bool SPLIT, int BN>
__global__ void __launch_bounds__(kTcThreads, 1)
largem_gemm_tc_kernel(const LargeMParams p, const __grid_constant__ CUtensorMap map_a,
                      const __grid_constant__ CUtensorMap map_alo, const __grid_constant__ CUtensorMap map_w) {
  using C = TcCfg<BN, SPLIT>;
  constexpr int STAGES = C::STAGES, STAGE_BYTES = C::STAGE_BYTES, B_BYTES = C::B_BYTES, OFF_BARS = C::OFF_BARS;
  constexpr int W_OFF = C::W_OFF;
  const uint32_t kIdesc = p.f16 ? C::IDESC_F16 : C::IDESC_BF16;
  constexpr int kTmemCols = 2 * BN;  // two fp32 accumulators of BN columns
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + OFF_BARS);
  uint64_t* empty = full + STAGES;
  uint64_t* tmem_full = empty + STAGES;
  uint64_t* tmem_empty = tmem_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + 2);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tiles_m = (p.M + BM - 1) / BM, tiles_n = (p.N + BN - 1) / BN;
  const int n_tiles = tiles_m * tiles_n;
  const int nkb = (p.K + BK - 1) / BK;

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&tmem_full[a], 1);
      mbar_init(&tmem_empty[a], 4);
    }
    fence_barrier_init();
  }
  if (warp == 1) {  // TMEM: 2 BN columns x 128 lanes of fp32
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "n"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_slot);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      bool ok = true;
      int it = 0;
      for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
        int tm, tn;
        tile_coords(t, tiles_m, tiles_n, tm, tn);
        const int m0 = tm * BM, n0 = tn * BN;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % STAGES;
          ok = mbar_wait_bounded(&empty[s], ((it / STAGES) & 1) ^ 1u);
          if (!ok) break;
          uint8_t* st = smem + s * STAGE_BYTES;
          mbar_expect_tx(&full[s], (SPLIT ? 2 : 1) * A_BYTES + B_BYTES);
          tma_load_2d(st, &map_a, kb * BK, m0, &full[s]);
          if (SPLIT) tma_load_2d(st + A_BYTES, &map_alo, kb * BK, m0, &full[s]);
          tma_load_2d(st + W_OFF, &map_w, kb * BK, n0, &full[s]);
        }
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
      int it = 0, i = 0;
      for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++i) {
        const int ab = i & 1;
        ok = mbar_wait_bounded(&tmem_empty[ab], ((i >> 1) & 1) ^ 1u);  // epilogue has drained this accumulator
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + ab * BN;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % STAGES;
          ok = mbar_wait_bounded(&full[s], (it / STAGES) & 1);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem + s * STAGE_BYTES);
          const uint64_t da = smem_desc(a_addr), dl = smem_desc(a_addr + A_BYTES), dw = smem_desc(a_addr + W_OFF);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)  // +32 bytes along K inside the swizzled row = +2 in the address field
            tc_mma(d_tmem, da + 2 * k, dw + 2 * k, kIdesc, (kb > 0 || k > 0) ? 1u : 0u);
          if (SPLIT) {
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k) tc_mma(d_tmem, dl + 2 * k, dw + 2 * k, kIdesc, 1u);
          }
          tc_commit(&empty[s]);  // the stage is free once these MMAs have read it
        }
        if (ok) tc_commit(&tmem_full[ab]);  // accumulator complete
      }
      if (!ok && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;  // the TMEM lane quarter this warp may access
    bool ok = true;
    int i = 0;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++i) {
      const int ab = i & 1;
      int tm, tn;
      tile_coords(t, tiles_m, tiles_n, tm, tn);
      const int m0 = tm * BM, n0 = tn * BN;
      if (ok) ok = mbar_wait_bounded(&tmem_full[ab], (i >> 1) & 1);
      if (!ok) break;
      tc_fence_after();
      const int m = m0 + q * 32 + lane;
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + ab * BN;
      for (int c = 0; c < BN; c += 32) {
        if (n0 + c >= p.N) break;  // uniform: the tile's tail columns do not exist
        uint32_t r[32];
        tc_ld32(taddr + c, r);
#pragma unroll
        for (int j = 0; j < 16; ++j)
          epilogue_pair(p, m, n0 + c + 2 * j, __uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tmem_empty[ab]);
    }
    if (!ok && lane == 0 && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------- host: tensor maps
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn g_encode = nullptr;

cudaError_t make_map(CUtensorMap* map, const void* base, int rows, int K, int box_rows, bool f16) {
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(K) * 2};
  const cuuint32_t box[2] = {BK, static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = g_encode(map, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

}  // namespace

cudaError_t largem_gemm_tc_init() {
  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    g_encode = reinterpret_cast<EncodeFn>(fn);
  }
  cudaError_t e = cudaFuncSetAttribute(largem_gemm_tc_kernel<true, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       TcCfg<256, true>::SMEM);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(largem_gemm_tc_kernel<false, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             TcCfg<256, false>::SMEM);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(largem_gemm_tc_kernel<true, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             TcCfg<128, true>::SMEM);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(largem_gemm_tc_kernel<false, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             TcCfg<128, false>::SMEM);
  return e;
}

namespace {
template <int BN>
cudaError_t launch_bn(const LargeMParams& p, cudaStream_t stream, int sm_count) {
  CUtensorMap ma, ml, mw;
  const bool f16 = p.f16 != 0;
  if (f16 && p.A_lo) return cudaErrorInvalidValue;  // the binary16 path takes one value per activation
  cudaError_t e = make_map(&ma, p.A, p.M, p.K, BM, f16);
  if (e == cudaSuccess) e = make_map(&ml, p.A_lo ? p.A_lo : p.A, p.M, p.K, BM, f16);
  if (e == cudaSuccess) e = make_map(&mw, p.W, p.N, p.K, BN, f16);
  if (e != cudaSuccess) return e;
  const int tiles = ((p.M + BM - 1) / BM) * ((p.N + BN - 1) / BN);
  const int grid = tiles < sm_count ? tiles : sm_count;
  if (p.A_lo) largem_gemm_tc_kernel<true, BN><<<grid, kTcThreads, TcCfg<BN, true>::SMEM, stream>>>(p, ma, ml, mw);
  else largem_gemm_tc_kernel<false, BN><<<grid, kTcThreads, TcCfg<BN, false>::SMEM, stream>>>(p, ma, ml, mw);
  return cudaGetLastError();
}
}  // namespace

cudaError_t launch_largem_gemm_tc(const LargeMParams& p, cudaStream_t stream, int sm_count) {
  if (!g_encode) return cudaErrorNotReady;
  if ((reinterpret_cast<uintptr_t>(p.A) | reinterpret_cast<uintptr_t>(p.W) | reinterpret_cast<uintptr_t>(p.A_lo)) & 15)
    return cudaErrorMisalignedAddress;
  // 256-wide tiles unless they leave SMs idle; then 128-wide ones (twice as many tiles)
  const int tiles256 = ((p.M + BM - 1) / BM) * ((p.N + 255) / 256);
  return tiles256 < sm_count ? launch_bn<128>(p, stream, sm_count) : launch_bn<256>(p, stream, sm_count);
}

}  // namespace ladder
