// Weight-streaming GEMM of the decode path for batch <= 4:  acc[b, n] = sum_k act[b, k] * W[n, k].
//
// HBM-bound by construction: every weight byte is read exactly once.  The rows of W are cut into
// 8-row units; persistent CTAs (one per SM) claim batches of consecutive units through an atomic
// claim counter and a fixed schedule -- 8 units (64 rows x all of K) while plenty is left,
// shrinking to 1-2 units towards the end (guided self-scheduling).  Dynamic claiming matters: under full load SMs stream
// at visibly different rates (measured spread ~15 %), and a static split makes every launch wait
// for the slowest SM.  A CTA has four roles that only meet at mbarriers:
//   * producer warp: claims batches (one at a time), publishes them through a shared-memory queue and
//     streams the batch's weights, K chunk by K chunk, as [8 rows x 2048 k] tiles -- eight 4 KB
//     bulk async copies (TMA engine, L2 evict-first) -- into a 4-stage ring.  4 KB segments are
//     what it takes to reach the read ceiling of the part (2 KB: ~5 % lower, 1 KB: half);
//   * four stager warps: turn the fp32 activations of the next K chunk into MMA operands:
//     (x * gain) as a bf16 high part plus a bf16 low part (x ~ hi + lo, ~16 mantissa bits).  The
//     high parts occupy columns 0-3 and the low parts columns 4-7 of ONE 8-column MMA tile, so the
//     extra precision costs no extra MMA (wider batches run on the tcgen05 kernel).  The
//     batches all walk the chunks in the same cyclic order, so the stagers free-run one chunk ahead.
//     They also form the RMSNorm sum of squares while staging the first batch's chunks;
//   * four consumer warps: split each tile along K, read 16 contiguous bytes of a weight row and
//     the matching 16 bytes of an activation row per thread (the K index inside an MMA is
//     permuted identically for both operands: no ldmatrix, no swizzle, conflict-free with a row
//     pitch of 64 mod 128 bytes) and issue mma.sync m16n8k16 with two consecutive 8-row stages as
//     the two row halves, software-pipelined so neither load nor MMA latency is exposed.
//     Activation fragments are hoisted into registers once per chunk; accumulators stay in
//     registers over the whole K.  The fragments of a finished batch go to a double-buffered
//     shared-memory slot and the warps move on;
//   * three finisher warps: add the four K-split fragments in a fixed order (deterministic), apply
//     1/rms and run the epilogue (residual add of Eq. 1 / Eq. 2, SwiGLU, rotary + KV append), off
//     the streaming path.
// Nothing before griddepcontrol.wait depends on the previous kernel (barrier set-up, claiming, the
// first ring fill), so under programmatic dependent launch the weight stream does not drain
// between kernels.
#include <algorithm>

#include "common.cuh"
#include "decode_schedule.h"
#include "kernels.h"
#include "smallm_epilogue.cuh"

namespace ladder {

// batch 9..64: tcgen05 kernel (default) or the earlier mma.sync kernel (cross-check)
cudaError_t launch_smallm_gemm_wide_tc(const SmallMParams& p, cudaStream_t stream, bool pdl, int sm_count);
cudaError_t launch_smallm_gemm_wide_stage(const SmallMParams& p, cudaStream_t stream, bool pdl);
cudaError_t smallm_gemm_wide_tc_init();
size_t smallm_gemm_wide_tc_smem_bytes(int batch);
size_t smallm_gemm_wide_tc_scratch_floats(int N, int K, int batch);
static int g_wide_impl = 0;  // 0 = tcgen05 kernel for batch > 4, 2 = tcgen05 kernel for every batch
void set_decode_wide_impl(int impl) { g_wide_impl = impl == 2 ? 2 : 0; }

namespace {

constexpr int kThreads = 384;  // warp 0 producer | warps 1-4 consumers | warps 5-8 stagers | warps 9-11 finishers
constexpr int kFin = 96;       // finisher threads
constexpr int TK = 2048;       // K elements per chunk (4 KB of a weight row)
constexpr int PITCH = TK * 2 + 64;
constexpr int STAGE_BYTES = 8 * PITCH;
constexpr int STAGES = 4;
constexpr int ACT_BYTES = 8 * PITCH;
constexpr int RG_MAX = kSchedUnitsMax / 2;  // 16-row groups per batch at most
static_assert(2 * RG_MAX == kSchedUnitsMax, "schedule and tile geometry disagree");
constexpr int SPW = TK / 32 / 4;    // 32-wide K slabs per consumer warp per chunk
constexpr int RED_FLOATS = 4 * RG_MAX * 4 * 32;
constexpr int QDEPTH = 16;          // claimed-item queue, producer -> consumers and finishers
constexpr int OFF_ACT = STAGES * STAGE_BYTES;
constexpr int OFF_SSQ = OFF_ACT + ACT_BYTES;      // [4 stager warps][8] sums of squares
constexpr int OFF_RED = OFF_SSQ + 4 * 8 * 4;
constexpr int OFF_RSTD = OFF_RED + 2 * RED_FLOATS * 4;  // two fragment slots
constexpr int OFF_BAR = OFF_RSTD + 8 * 4;  // full[4], empty[4], act_free, act_full, norm_ready, red_full[2], red_free[2]
constexpr int OFF_MISC = OFF_BAR + (2 * STAGES + 7) * 8;  // queue[QDEPTH], q_head, act_want, flag, last
constexpr int SMEM = OFF_MISC + (QDEPTH + 4) * 4 + 16 + 128;
static_assert(SMEM <= 190 * 1024, "leave room for a co-resident attention CTA");

struct F8 {
  float4 a, b;
};

// bounded spin on a shared-memory counter written by another warp of this CTA
__device__ __forceinline__ bool wait_counter_gt(const volatile int* ctr, int n) {
  if (*ctr > n) return true;
  const long long t0 = clock64();
  for (uint32_t i = 1;; ++i) {
    if (*ctr > n) return true;
    if ((i & 255u) == 0 && clock64() - t0 > kWaitCycles) return false;
  }
}

// bounded mbarrier wait that also gives up when a shared-memory stop flag goes negative:
// 0 = phase completed, 1 = stop flag seen, 2 = timed out
__device__ __forceinline__ int mbar_wait_or_stop(uint64_t* bar, uint32_t parity, const volatile int* stop) {
  const long long t0 = clock64();
  for (uint32_t i = 1;; ++i) {
    if (mbar_try_wait(bar, parity)) return 0;
    if (*stop < 0) return 1;
    if ((i & 255u) == 0 && clock64() - t0 > kWaitCycles) return 2;
  }
}

// One [16 rows x 2048 k] tile of a consumer warp: its SPW 32-wide K slabs, two 8-row stages as the two
// row halves of the MMA, software-pipelined over groups of 2 slabs (the shared-memory loads of group
// i+1 are issued before the MMAs of group i), two accumulator chains.  FAST: every slab lies inside K
// and both stages are present, so nothing is predicated.
template <bool FAST>
__device__ __forceinline__ void slab_loop(float (&acc0)[4], float (&acc1)[4], const uint4 (&bf)[SPW], uint32_t base0,
                                          uint32_t base1, int cw, int k0, int K, int tig, bool hi_valid) {
  uint4 lo[2][2], hi[2][2];
  auto load_group = [&](int grp, uint4(&l)[2], uint4(&h)[2]) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int slab = cw * SPW + grp * 2 + e;
      if (FAST) {
        l[e] = lds128(base0 + slab * 64);
        h[e] = lds128(base1 + slab * 64);
      } else {
        const bool kv = (k0 + slab * 32 + tig * 8) < K;
        l[e] = make_uint4(0, 0, 0, 0);
        h[e] = make_uint4(0, 0, 0, 0);
        if (kv) l[e] = lds128(base0 + slab * 64);
        if (kv && hi_valid) h[e] = lds128(base1 + slab * 64);
      }
    }
  };
  load_group(0, lo[0], hi[0]);
#pragma unroll
  for (int grp = 0; grp < SPW / 2; ++grp) {
    if (grp + 1 < SPW / 2) load_group(grp + 1, lo[(grp + 1) & 1], hi[(grp + 1) & 1]);
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int j = grp * 2 + e;
      const uint4& l = lo[grp & 1][e];
      const uint4& h = hi[grp & 1][e];
      mma_bf16_16816(acc0, l.x, h.x, l.y, h.y, bf[j].x, bf[j].y);
      mma_bf16_16816(acc1, l.z, h.z, l.w, h.w, bf[j].z, bf[j].w);
    }
  }
}


template <bool NORM>
__global__ void __launch_bounds__(kThreads, 1) decode_gemm_kernel(const SmallMParams p, const Schedule sched) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  uint8_t* ring = smem;
  uint8_t* act = smem + OFF_ACT;
  float* ssq_part = reinterpret_cast<float*>(smem + OFF_SSQ);
  float* red = reinterpret_cast<float*>(smem + OFF_RED);
  float* rstd_s = reinterpret_cast<float*>(smem + OFF_RSTD);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
  uint64_t* empty = full + STAGES;
  uint64_t* act_free = empty + STAGES;
  uint64_t* act_full = act_free + 1;
  uint64_t* norm_ready = act_full + 1;
  uint64_t* red_full = norm_ready + 1;   // [2] consumers -> finishers
  uint64_t* red_free = red_full + 2;     // [2] finishers -> consumers
  int* queue = reinterpret_cast<int*>(smem + OFF_MISC);
  volatile int* q_head = queue + QDEPTH;
  volatile int* act_want = queue + QDEPTH + 1;
  int* flag_s = queue + QDEPTH + 2;
  int* last_s = queue + QDEPTH + 3;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int batch = p.batch;
  const int nchunk = (p.K + TK - 1) / TK;
  const int n_units = p.N >> 3;  // 8-row units

  if (tid == 0) {
    int dead = 0;
    if (p.status) dead = (*reinterpret_cast<volatile int32_t*>(p.status) & LADDER_DEV_TIMEOUT) ? 1 : 0;
    *flag_s = dead;
    *q_head = 0;
    *act_want = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 4);
    }
    mbar_init(act_free, 4);
    mbar_init(act_full, 4);
    mbar_init(norm_ready, 4);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&red_full[s], 4);
      mbar_init(&red_free[s], 3);
    }
    fence_barrier_init();
  }
  __syncthreads();
  pdl_launch_dependents();
  if (*flag_s) return;  // an earlier kernel reported a protocol error: do nothing

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    const uint64_t pol = l2_policy_evict_first();
    const uint8_t* Wb = reinterpret_cast<const uint8_t*>(p.W);
    bool ok = true;
    int it = 0, n = 0;
    int c = 0;
    while (ok) {
      // one claim at a time (claiming ahead would let a CTA hoard batches it cannot start yet);
      // the round trip is covered by the weights already in the ring
      int u0 = 0, nu = 0;
      if (lane == 0) {
        c = atomicAdd(p.work, 1);
        int ci = c, ubase = 0;
        for (int ph = 0; ph < sched.n; ++ph) {  // claim index -> (first unit, units) by the fixed schedule
          if (ci < sched.count[ph]) {
            u0 = ubase + ci * sched.size[ph];
            nu = min(sched.size[ph], n_units - u0);
            break;
          }
          ci -= sched.count[ph];
          ubase += sched.count[ph] * sched.size[ph];
        }
        queue[n % QDEPTH] = nu > 0 ? (u0 * 16 + nu) : -1;
        __threadfence_block();
        *q_head = n + 1;
      }
      ++n;
      u0 = __shfl_sync(0xffffffffu, u0, 0);
      nu = __shfl_sync(0xffffffffu, nu, 0);
      if (nu == 0) break;
      const int row0 = u0 * 8;
      for (int ch = 0; ch < nchunk && ok; ++ch) {
        const int k0 = ch * TK;
        const uint32_t kb = static_cast<uint32_t>(min(TK, p.K - k0)) * 2u;
        for (int h8 = 0; h8 < nu; ++h8) {
          const int st = it % STAGES;
          ok = mbar_wait_bounded(&empty[st], ((it / STAGES) & 1) ^ 1u);
          if (!ok) break;
          if (lane == 0) mbar_expect_tx(&full[st], 8 * kb);
          __syncwarp();
          if (lane < 8) {
            const size_t row = static_cast<size_t>(row0 + h8 * 8 + lane);
            bulk_g2s(ring + st * STAGE_BYTES + lane * PITCH, Wb + (row * p.K + k0) * 2, kb, &full[st], pol);
          }
          ++it;
        }
      }
    }
    if (!ok) {
      // protocol error: record it, stop the consumers, wait (bounded) for the copies in flight
      if (lane == 0) {
        if (p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
        queue[n % QDEPTH] = -1;
        __threadfence_block();
        *q_head = n + 1;
      }
      for (int j = 1; j <= STAGES && j <= it; ++j) {
        const int i2 = it - j;
        mbar_wait_bounded(&full[i2 % STAGES], (i2 / STAGES) & 1);
      }
    }
    // the last CTA to run out of work rewinds the claim counter for the next use of this slot
    if (lane == 0) {
      const int d = atomicAdd(p.work + 1, c >= 0 ? 1 : 2);  // ordered after the last claim's return
      if (d == static_cast<int>(gridDim.x) - 1) {
        p.work[0] = 0;
        p.work[1] = 0;
      }
    }
    return;
  }

  if (warp >= 5 && warp < 9) {
    // ------------------------------------------------------------------ stagers
    const int st = tid - 160;  // 0..127
    const int sw = warp - 5;
    const uint32_t act_u32 = smem_u32(act);
    const float* actf = static_cast<const float*>(p.act);
    bool ok = true;
    pdl_wait();  // activations come from the previous kernel

    // RMSNorm: the sum of squares of every activation row is accumulated while the chunks of the
    // FIRST batch are staged (they cover the whole K once); no separate pass over x.
    float ssq[8];
#pragma unroll
    for (int b = 0; b < 8; ++b) ssq[b] = 0.f;
    bool ssq_on = NORM;

    F8 x[4][2];
    uint4 gq[2];
    bool kv[2];
    auto load_rows = [&](int ch, int round) {
      const int k0 = ch * TK;
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int k = k0 + (st + u * 128) * 8;
        kv[u] = k < p.K;
        gq[u] = make_uint4(0x3f803f80u, 0x3f803f80u, 0x3f803f80u, 0x3f803f80u);  // gain 1.0
        if (NORM) gq[u] = kv[u] ? __ldg(reinterpret_cast<const uint4*>(p.gain + k)) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int b = round * 4 + i;
          x[i][u].a = x[i][u].b = make_float4(0, 0, 0, 0);
          if (kv[u] && b < batch) {
            const float4* src =
                reinterpret_cast<const float4*>(actf + static_cast<size_t>(b) * p.K + k0 + (st + u * 128) * 8);
            x[i][u].a = src[0];
            x[i][u].b = src[1];
          }
        }
    };
    auto store_rows = [&](int round) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int b = round * 4 + i;
        if (b >= batch) break;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          float y[8] = {x[i][u].a.x, x[i][u].a.y, x[i][u].a.z, x[i][u].a.w,
                        x[i][u].b.x, x[i][u].b.y, x[i][u].b.z, x[i][u].b.w};
          if (NORM) {
            if (ssq_on)
              ssq[b] += y[0] * y[0] + y[1] * y[1] + y[2] * y[2] + y[3] * y[3] + y[4] * y[4] + y[5] * y[5] +
                        y[6] * y[6] + y[7] * y[7];
            y[0] *= bf16_lo(gq[u].x);
            y[1] *= bf16_hi(gq[u].x);
            y[2] *= bf16_lo(gq[u].y);
            y[3] *= bf16_hi(gq[u].y);
            y[4] *= bf16_lo(gq[u].z);
            y[5] *= bf16_hi(gq[u].z);
            y[6] *= bf16_lo(gq[u].w);
            y[7] *= bf16_hi(gq[u].w);
          }
          uint4 hi;
          hi.x = pack_bf16x2(y[0], y[1]);
          hi.y = pack_bf16x2(y[2], y[3]);
          hi.z = pack_bf16x2(y[4], y[5]);
          hi.w = pack_bf16x2(y[6], y[7]);
          const uint32_t dst = act_u32 + b * PITCH + (st + u * 128) * 16;
          sts128(dst, hi);
          uint4 lo;
          lo.x = pack_bf16x2(y[0] - bf16_lo(hi.x), y[1] - bf16_hi(hi.x));
          lo.y = pack_bf16x2(y[2] - bf16_lo(hi.y), y[3] - bf16_hi(hi.y));
          lo.z = pack_bf16x2(y[4] - bf16_lo(hi.z), y[5] - bf16_hi(hi.z));
          lo.w = pack_bf16x2(y[6] - bf16_lo(hi.w), y[7] - bf16_hi(hi.w));
          sts128(dst + 4 * PITCH, lo);
        }
      }
    };

    // Every batch walks the chunks 0 .. nchunk-1, so the stagers free-run through that cyclic
    // sequence one chunk ahead of the consumers: chunk r is written as soon as chunk r-1 has been
    // hoisted (act_free), its raw values having been loaded into registers before that.
    for (int r = 0;; ++r) {
      const int ch = r % nchunk;
      load_rows(ch, 0);
      const int w = mbar_wait_or_stop(act_free, (r & 1) ^ 1u, act_want);
      if (w == 2) ok = false;
      if (w != 0) break;  // the consumers have run out of work (or a protocol error)
      store_rows(0);
      if (NORM && r == nchunk - 1) {  // every chunk has been staged once: publish the sums
#pragma unroll
        for (int b = 0; b < 8; ++b) {
          if (b >= batch) break;
          const float t = warp_sum(ssq[b]);
          if (lane == 0) ssq_part[sw * 8 + b] = t;
        }
        ssq_on = false;
        __syncwarp();
        if (lane == 0) mbar_arrive(norm_ready);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(act_full);
    }
    if (!ok && lane == 0 && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
    return;
  }

  if (warp >= 9) {
    // ------------------------------------------------------------------ finishers
    const int ft = tid - 288;  // 0..95
    bool ok = true;
    pdl_wait();  // the addend of the residual epilogue comes from the previous kernel
    bool have_rstd = !NORM;
    auto need_rstd = [&]() {  // 1/rms of every activation row, once per CTA (uniform call sites)
      if (have_rstd) return;
      if (ok) ok = mbar_wait_bounded(norm_ready, 0);
      if (ft < batch) {
        const float s = ssq_part[ft] + ssq_part[8 + ft] + ssq_part[16 + ft] + ssq_part[24 + ft];
        rstd_s[ft] = rsqrtf(s / static_cast<float>(p.K) + p.eps);
      }
      asm volatile("bar.sync 2, 96;" ::: "memory");
      have_rstd = true;
    };
    for (int n = 0;; ++n) {
      if (ok) ok = wait_counter_gt(q_head, n);
      const int id = ok ? reinterpret_cast<volatile int*>(queue)[n % QDEPTH] : -1;
      if (id < 0) break;
      const int row0 = (id >> 4) * 8, rows = (id & 15) * 8;
      const int slot = n & 1;
      if (ok) ok = mbar_wait_bounded(&red_full[slot], (n >> 1) & 1);
      const float* rs = red + slot * RED_FLOATS;
      auto column = [&](int a, int rr, int c) -> float {
        const int idx = (a * 4 + ((rr >> 3) * 2 + (c & 1))) * 32 + ((rr & 7) * 4 + (c >> 1));
        return rs[idx] + rs[RG_MAX * 128 + idx] + rs[2 * RG_MAX * 128 + idx] + rs[3 * RG_MAX * 128 + idx];
      };
      need_rstd();
      auto value = [&](int r, int b) -> float {
        const int a = r >> 4, rr = r & 15;
        float s = column(a, rr, b);
        s += column(a, rr, b + 4);  // high-part product + low-part product
        if (NORM) s *= rstd_s[b];
        return s;
      };
      smallm_epilogue<kFin>(p, ft, rows, row0, batch, value);
      __syncwarp();
      if (lane == 0) mbar_arrive(&red_free[slot]);  // the consumers may refill this slot
    }
    if (!ok && lane == 0 && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
    return;
  }

  // -------------------------------------------------------------------- consumers
  const int ct = tid - 32;  // 0..127
  const int cw = warp - 1;  // 0..3
  const int g = lane >> 2, tig = lane & 3;
  const uint32_t ring_u32 = smem_u32(ring);
  const uint32_t act_u32 = smem_u32(act);
  // which activation row feeds MMA column g: packed = hi rows 0-3 then lo rows 4-7 of batch g & 3
  const bool col_valid = (g & 3) < batch;
  bool ok = true;

  uint4 bf[SPW];
#pragma unroll
  for (int j = 0; j < SPW; ++j) bf[j] = make_uint4(0, 0, 0, 0);
  int it = 0, n_req = 0;
  for (int n = 0;; ++n) {
    if (ok) ok = wait_counter_gt(q_head, n);
    const int id = ok ? reinterpret_cast<volatile int*>(queue)[n % QDEPTH] : -1;
    if (id < 0) break;
    const int rows = (id & 15) * 8;
    const int rgn = (rows + 15) >> 4;

    float acc[RG_MAX][2][4];
#pragma unroll
    for (int a = 0; a < RG_MAX; ++a)
#pragma unroll
      for (int q = 0; q < 2; ++q)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[a][q][c] = 0.f;

    for (int ch = 0; ch < nchunk; ++ch) {
      const int k0 = ch * TK;
      // hoist this warp's activation fragments of the chunk, then hand the buffer back
      if (ok) ok = mbar_wait_bounded(act_full, n_req & 1);
      ++n_req;
#pragma unroll
      for (int j = 0; j < SPW; ++j) bf[j] = lds128(act_u32 + g * PITCH + (cw * SPW + j) * 64 + tig * 16);
      if (!col_valid) {  // rows of the buffer beyond the batch hold stale data: their MMA columns are zeroed
#pragma unroll
        for (int j = 0; j < SPW; ++j) bf[j] = make_uint4(0, 0, 0, 0);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(act_free);
#pragma unroll
      for (int rgi = 0; rgi < RG_MAX; ++rgi) {
        if (rgi >= rgn) break;  // uniform across the CTA
        const bool hi_valid = (rgi * 16 + 8) < rows;
        const int st0 = it % STAGES, st1 = (it + 1) % STAGES;
        if (ok) ok = mbar_wait_bounded(&full[st0], (it / STAGES) & 1);
        if (ok && hi_valid) ok = mbar_wait_bounded(&full[st1], ((it + 1) / STAGES) & 1);
        const uint32_t base0 = ring_u32 + st0 * STAGE_BYTES + g * PITCH + tig * 16;
        const uint32_t base1 = ring_u32 + st1 * STAGE_BYTES + g * PITCH + tig * 16;
        // a full chunk with both 8-row halves present (the common case) takes the path without
        // predicates: a guarded shared-memory load compiles to a branch, and 64 of them per tile
        // cost more than the loads and MMAs themselves
        if (hi_valid && k0 + TK <= p.K) slab_loop<true>(acc[rgi][0], acc[rgi][1], bf, base0, base1, cw, k0, p.K, tig, true);
        else slab_loop<false>(acc[rgi][0], acc[rgi][1], bf, base0, base1, cw, k0, p.K, tig, hi_valid);
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(&empty[st0]);
          if (hi_valid) mbar_arrive(&empty[st1]);
        }
        it += hi_valid ? 2 : 1;
      }
    }

    // hand the accumulator fragments to the finishers and move on
    const int slot = n & 1;
    if (ok) ok = mbar_wait_bounded(&red_free[slot], ((n >> 1) & 1) ^ 1u);
    float* rs = red + slot * RED_FLOATS;
#pragma unroll
    for (int a = 0; a < RG_MAX; ++a) {
      if (a >= rgn) break;
#pragma unroll
      for (int c = 0; c < 4; ++c) rs[((cw * RG_MAX + a) * 4 + c) * 32 + lane] = acc[a][0][c] + acc[a][1][c];
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&red_full[slot]);
  }
  // release the stagers (they are waiting for the hand-back of a chunk nobody will use)
  if (ct == 0) *act_want = -1;
  if (!ok && lane == 0 && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
}

cudaError_t launch_small(const SmallMParams& p, cudaStream_t stream, bool pdl, int grid) {
  auto kern = p.act_mode == ACT_F32_NORM ? decode_gemm_kernel<true> : decode_gemm_kernel<false>;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = SMEM;
  cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  const Schedule sc = make_schedule(p.N >> 3, grid);
  return cudaLaunchKernelEx(&cfg, kern, p, sc);
}

}  // namespace


cudaError_t smallm_gemm_init() {
  cudaError_t e = cudaFuncSetAttribute(decode_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(decode_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
  if (e == cudaSuccess) e = smallm_gemm_wide_tc_init();
  return e;
}

size_t smallm_gemm_smem_bytes(int batch) {
  if (batch <= 4) return SMEM;
  const size_t wide = smallm_gemm_wide_tc_smem_bytes(batch);
  return std::max(wide, static_cast<size_t>(SMEM));
}

size_t smallm_gemm_scratch_floats(int N, int K, int batch) {
  return smallm_gemm_wide_tc_scratch_floats(N, K, batch);  // staged activations + shared-tile pieces
}

cudaError_t launch_smallm_gemm_stage(const SmallMParams& p, cudaStream_t stream, bool pdl) {
  if (p.batch <= 4 && g_wide_impl != 2 && !p.force_wide) return cudaErrorInvalidValue;  // the batch <= 4 kernel stages inside itself
  return launch_smallm_gemm_wide_stage(p, stream, pdl);
}

cudaError_t launch_smallm_gemm(const SmallMParams& p, cudaStream_t stream, bool pdl, int sm_count) {
  // Batch 5..64 on the tcgen05 kernel: this file's kernel holds a bf16 hi + lo activation pair only for batch <= 4
  // (one 8-column MMA tile).
  if (p.batch > 4 || g_wide_impl == 2 || p.force_wide) return launch_smallm_gemm_wide_tc(p, stream, pdl, sm_count);
  if (!p.work || p.act_pending || p.act_pending2 || p.act_sum_out || p.wide_prestaged) return cudaErrorInvalidValue;
  const int units = p.N >> 3;
  const int grid = units < sm_count ? units : sm_count;
  return launch_small(p, stream, pdl, grid);
}

}  // namespace ladder
