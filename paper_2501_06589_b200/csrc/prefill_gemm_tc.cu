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

// ---------------------------------------------------------------- CTA pairs (cta_group::2)
// The same GEMM with 256 x 256 output tiles computed by a PAIR of CTAs on neighbouring SMs (a cluster of two):
// every CTA stages its own 128 rows of A and its own 128 of the tile's 256 W rows, and the leader's MMA thread issues
// tcgen05.mma.cta_group::2 (M 256, N 256, K 16), which reads both CTAs' shared memory and writes 128 accumulator
// rows into each CTA's tensor memory.  Per MMA a CTA's shared memory now supplies 8 KB instead of 12 KB and per K
// block takes in 32 KB instead of 48 KB: with one CTA per tile the operand traffic (reads by the tensor core plus
// writes by the TMA unit) exceeds what shared memory delivers per cycle, which is what held that kernel near 70 %
// of the tensor rate.  Single-value operands only (binary16, or one bf16 value per activation).
//   warp 0   TMA producer in BOTH CTAs; the copies of both complete on the LEADER's full barrier (the leader
//            announces the bytes of both); no multicast: each CTA fetches only what it alone needs;
//   warp 1   leader: the MMA issuer; tcgen05.commit arrives on the ring's empty barriers and on the accumulator-full
//            barriers of BOTH CTAs.  In both CTAs this warp owns the (paired) TMEM allocation;
//   warps 2-5 epilogue of the CTA's own 128 rows; all eight epilogue warps of the pair release an accumulator on
//            the leader's barrier.
// The pair meets at a cluster barrier after set-up and before the tensor memory is freed.  Every wait is bounded.
constexpr int P2_STAGES = 6, P2_A_BYTES = 128 * BK * 2, P2_STAGE_BYTES = 2 * P2_A_BYTES;  // A half + W half: 32 KB
constexpr int P2_OFF_BARS = P2_STAGES * P2_STAGE_BYTES;
constexpr int P2_SMEM = P2_OFF_BARS + 24 * 8 + 1024;
constexpr int P2_BN = 256, P2_BM = 256, P2_GROUP_M = 8;  // bands of 8 x 256 rows (4 and 16 measured slower)
constexpr uint32_t P2_IDESC_F16 = (1u << 4) | (static_cast<uint32_t>(P2_BN >> 3) << 17) |
                                  (static_cast<uint32_t>(P2_BM >> 4) << 24);
constexpr uint32_t P2_IDESC_BF16 = P2_IDESC_F16 | (1u << 7) | (1u << 10);

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// the address of this CTA's shared-memory location `addr` as seen in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// 2-D tile into this CTA's shared memory; completes on a barrier that may live in the peer CTA
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(bar_cluster), "r"(x), "r"(y)
      : "memory");
}
// arrives (once all MMAs issued so far have completed) on the barrier at this offset in BOTH CTAs of the pair
__device__ __forceinline__ void tc_commit_pair(uint64_t* bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"(mask)
               : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc)
      : "memory");
}

__global__ void __launch_bounds__(kTcThreads, 1)
largem_gemm_tc_pair_kernel(const LargeMParams p, const __grid_constant__ CUtensorMap map_a,
                           const __grid_constant__ CUtensorMap map_w) {
  const uint32_t kIdesc = p.f16 ? P2_IDESC_F16 : P2_IDESC_BF16;
  constexpr int kTmemCols = 2 * P2_BN;  // two fp32 accumulators of 256 columns (128 rows of them in each CTA)
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + P2_OFF_BARS);
  uint64_t* empty = full + P2_STAGES;
  uint64_t* tmem_full = empty + P2_STAGES;
  uint64_t* tmem_empty = tmem_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + 2);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = leader
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int tiles_m = (p.M + P2_BM - 1) / P2_BM, tiles_n = (p.N + P2_BN - 1) / P2_BN;
  const int n_tiles = tiles_m * tiles_n;
  const int nkb = (p.K + BK - 1) / BK;
  auto coords = [&](int t, int& tm, int& tn) {  // bands of P2_GROUP_M m-tiles, m fastest inside a band
    const int per_band = P2_GROUP_M * tiles_n;
    const int band = t / per_band, r = t - band * per_band;
    const int m_first = band * P2_GROUP_M;
    const int band_m = min(P2_GROUP_M, tiles_m - m_first);
    tm = m_first + r % band_m;
    tn = r / band_m;
  };

  if (tid == 0) {
    for (int s = 0; s < P2_STAGES; ++s) {
      mbar_init(&full[s], 1);   // used in the leader: its producer's arrive + the bytes of both CTAs
      mbar_init(&empty[s], 1);  // one commit
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&tmem_full[a], 1);
      mbar_init(&tmem_empty[a], 8);  // used in the leader: four epilogue warps of each CTA
    }
    fence_barrier_init();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "n"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers are initialised and its tensor memory allocated
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_slot);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      bool ok = true;
      int it = 0;
      for (int t = pair; t < n_tiles && ok; t += n_pairs) {
        int tm, tn;
        coords(t, tm, tn);
        const int m0 = tm * P2_BM + static_cast<int>(rank) * 128, n0 = tn * P2_BN + static_cast<int>(rank) * 128;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % P2_STAGES;
          ok = mbar_wait_bounded(&empty[s], ((it / P2_STAGES) & 1) ^ 1u);
          if (!ok) break;
          uint8_t* st = smem + s * P2_STAGE_BYTES;
          const uint32_t bar = mapa_u32(smem_u32(&full[s]), 0);  // the leader's barrier
          if (rank == 0) mbar_expect_tx(&full[s], 2 * P2_STAGE_BYTES);
          tma_load_2d_pair(st, &map_a, kb * BK, m0, bar);
          tma_load_2d_pair(st + P2_A_BYTES, &map_w, kb * BK, n0, bar);
        }
      }
      if (!ok) {
        if (p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
        const long long t0 = clock64();  // copies still in flight land in this CTA's shared memory: let them
        while (clock64() - t0 < 200000ll) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader only)
    if (lane == 0 && rank == 0) {
      bool ok = true;
      int it = 0, i = 0;
      for (int t = pair; t < n_tiles && ok; t += n_pairs, ++i) {
        const int ab = i & 1;
        ok = mbar_wait_bounded(&tmem_empty[ab], ((i >> 1) & 1) ^ 1u);  // both epilogues have drained this accumulator
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + ab * P2_BN;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % P2_STAGES;
          ok = mbar_wait_bounded(&full[s], (it / P2_STAGES) & 1);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem + s * P2_STAGE_BYTES);
          const uint64_t da = smem_desc(a_addr), dw = smem_desc(a_addr + P2_A_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            tc_mma_pair(d_tmem, da + 2 * k, dw + 2 * k, kIdesc, (kb > 0 || k > 0) ? 1u : 0u);
          tc_commit_pair(&empty[s]);  // the stage is free in both CTAs once these MMAs have read it
        }
        if (ok) tc_commit_pair(&tmem_full[ab]);  // accumulator complete, in both CTAs
      }
      if (!ok && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
    const int q = warp & 3;  // the TMEM lane quarter this warp may access
    bool ok = true;
    int i = 0;
    for (int t = pair; t < n_tiles; t += n_pairs, ++i) {
      const int ab = i & 1;
      int tm, tn;
      coords(t, tm, tn);
      const int m0 = tm * P2_BM + static_cast<int>(rank) * 128, n0 = tn * P2_BN;
      if (ok) ok = mbar_wait_bounded(&tmem_full[ab], (i >> 1) & 1);
      if (!ok) break;
      tc_fence_after();
      const int m = m0 + q * 32 + lane;
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + ab * P2_BN;
      for (int c = 0; c < P2_BN; c += 32) {
        if (n0 + c >= p.N) break;  // uniform: the tile's tail columns do not exist
        uint32_t r[32];
        tc_ld32(taddr + c, r);
#pragma unroll
        for (int j = 0; j < 16; ++j)
          epilogue_pair(p, m, n0 + c + 2 * j, __uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa_u32(smem_u32(&tmem_empty[ab]), 0));
    }
    if (!ok && lane == 0 && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // nobody in the pair reads the other's shared or tensor memory any more
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(kTmemCols) : "memory");
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
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(largem_gemm_tc_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, P2_SMEM);
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

namespace {
int g_prefill_impl = 0;
int g_sm_count = 0;
bool g_pair_tiles = true;  // 256 x 256 tiles on CTA pairs where the operands are single values and tiles are plenty

// CTA pairs: grid = 2 x min(pairs of SMs, tiles), launched as clusters of two
cudaError_t launch_pair(const LargeMParams& p, cudaStream_t stream, int sm_count) {
  CUtensorMap ma, mw;
  const bool f16 = p.f16 != 0;
  cudaError_t e = make_map(&ma, p.A, p.M, p.K, 128, f16);
  if (e == cudaSuccess) e = make_map(&mw, p.W, p.N, p.K, 128, f16);
  if (e != cudaSuccess) return e;
  const int tiles = ((p.M + P2_BM - 1) / P2_BM) * ((p.N + P2_BN - 1) / P2_BN);
  const int pairs = tiles < sm_count / 2 ? tiles : sm_count / 2;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = P2_SMEM;
  cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 2;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, largem_gemm_tc_pair_kernel, p, ma, mw);
}
}  // namespace

// 4 = the default operand formats with one CTA per tile everywhere (A/B measurements of the CTA-pair kernel)
void set_prefill_gemm_impl(int impl) {
  g_pair_tiles = impl != 4;
  g_prefill_impl = impl == 2 || impl == 3 ? impl : 0;
}
bool prefill_single_bf16() { return g_prefill_impl == 2; }
int prefill_gemm_impl() { return g_prefill_impl; }

cudaError_t launch_largem_gemm(const LargeMParams& p, cudaStream_t stream) {
  if (!g_sm_count) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&g_sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      g_sm_count = 148;
  }
  return launch_largem_gemm_tc(p, stream, g_sm_count);
}

cudaError_t launch_largem_gemm_tc(const LargeMParams& p, cudaStream_t stream, int sm_count) {
  if (!g_encode) return cudaErrorNotReady;
  if ((reinterpret_cast<uintptr_t>(p.A) | reinterpret_cast<uintptr_t>(p.W) | reinterpret_cast<uintptr_t>(p.A_lo)) & 15)
    return cudaErrorMisalignedAddress;
  // single-value operands and at least one 256 x 256 tile per pair of SMs: CTA pairs
  const int tiles_pair = ((p.M + P2_BM - 1) / P2_BM) * ((p.N + P2_BN - 1) / P2_BN);
  if (g_pair_tiles && !p.A_lo && tiles_pair >= sm_count / 2) return launch_pair(p, stream, sm_count);
  // 256-wide tiles unless they leave SMs idle; then 128-wide ones (twice as many tiles)
  const int tiles256 = ((p.M + BM - 1) / BM) * ((p.N + 255) / 256);
  return tiles256 < sm_count ? launch_bn<128>(p, stream, sm_count) : launch_bn<256>(p, stream, sm_count);
}

}  // namespace ladder
