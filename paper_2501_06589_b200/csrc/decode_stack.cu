// Persistent layer-stack kernel of the decode step (batch <= 8).
//
// One cooperative launch, one CTA per SM, runs EVERY weight-streaming GEMM of a decode step (QKV,
// Wo, gate/up, down of each layer and the LM head) plus the attention of every layer.  The GEMMs are
// "phases" walked in a fixed order by all CTAs; inside a phase the 8-row units of W are handed out in
// batches: whole rounds of one batch per CTA statically (batch i to CTA i mod grid), the short batches
// at the end of a long phase through an atomic counter.  What used to be a kernel boundary is a counter
// in global memory (units finished per phase): a reader polls it, with an acquire load and a time
// limit, only before it touches data another SM produced.
//
// Why: the weight stream of a phase depends on nothing, so the producer warp runs through phase
// after phase and the TMA ring never drains, whatever the consumers are waiting for.  With the
// ladder recurrence (Eq. 2) the input of a module is x_{m-2}: in the order
//     QKV_l, gate/up_l, Wo_l, down_l, QKV_{l+1}, ...
// every dependency points at least two phases back, so the polls succeed at once, and the
// attention of layer l (dedicated warps of the same CTAs) has the whole gate/up phase to finish
// before Wo_l needs it.  This is the paper's decoupling of a module from its predecessor's
// synchronisation, applied to the grid-wide hand-over inside one GPU instead of the all-reduce
// between GPUs.  Standard-residual layers (Eq. 1) run QKV, Wo, gate/up, down with every phase
// depending on the one before: correct, but the consumers stall at each hand-over.
//
// Warp roles (512 threads, four warpgroups so that registers can be moved between them):
//   warp 0        producer: claims batches, publishes them in a shared-memory queue, streams the
//                 weights as [8 rows x 2048 k] tiles (eight 4 KB bulk async copies) into a 5-stage ring
//   warps 1-3     finishers: K-split reduction, 1/rms, epilogue (residual add / SwiGLU / rotary + KV
//                 append), then publish the finished units (fence + release add)
//   warps 4-7     consumers: mma.sync m16n8k16 with the weights as the A operand (see decode_gemm.cu)
//   warps 8-11    stagers: the MMA operand form of the activations (bf16 hi + lo), one chunk ahead: copied
//                 when the phase that produced them wrote that form too (its epilogue does, with this
//                 phase's RMSNorm gain folded in), else converted from fp32; RMSNorm sum of squares from
//                 the fp32 rows while the first batch of a phase is staged
//   warps 12-15   attention: split-KV partials (64 keys x head group x sequence per unit), then the
//                 log-sum-exp merge, units dealt round-robin over the CTAs
// Data produced inside the launch is always read through L2 (ld.global.cg / acquire), never through
// the non-coherent L1 path and never by the TMA engine (a bulk copy of bytes other SMs had just written
// returned stale data now and then, proxy fences on both sides notwithstanding).  Every wait is bounded (about 0.3 s) and also gives up when another CTA has
// reported a timeout in the device status word, so a protocol error ends the launch quickly with
// LADDER_DEV_TIMEOUT set instead of hanging the device.
#include "common.cuh"
#include "kernels.h"
#include "smallm_epilogue.cuh"

namespace ladder {
namespace {

constexpr int kThreads = 512;
constexpr int kFin = 96;  // finisher threads
constexpr int kAux = 128;  // attention threads
constexpr int TK = kStackChunkK;   // K elements per chunk
constexpr int PITCH = TK * 2 + 64;
constexpr int STAGE_BYTES = 8 * PITCH;
constexpr int STAGES = 5;  // odd is fine: tiles are consumed as pairs of consecutive ring slots
constexpr int ACT_BYTES = 8 * PITCH;
constexpr int RG_MAX = kSchedUnitsMax / 2;
static_assert(2 * RG_MAX == kSchedUnitsMax, "schedule and tile geometry disagree");
constexpr int SPW = TK / 32 / 4;
constexpr int RED_FLOATS = 4 * RG_MAX * 4 * 32;
constexpr int QDEPTH = 16;
constexpr int NORM_RING = 4;  // the stagers run at most three normalised phases ahead of the finishers
constexpr int kChunk = 64;         // keys per attention unit
constexpr int kMaxSplits = 1024;   // merge weights held in shared memory

constexpr int OFF_ACT = STAGES * STAGE_BYTES;
constexpr int OFF_SSQ = OFF_ACT + ACT_BYTES;                 // [NORM_RING][4 stager warps][8]
constexpr int OFF_RED = OFF_SSQ + NORM_RING * 4 * 8 * 4;
constexpr int OFF_RSTD = OFF_RED + 2 * RED_FLOATS * 4;
constexpr int N_BARS = 2 * STAGES + 2 + NORM_RING + 4;       // full, empty, act_free, act_full, norm_ready[], red_full[2], red_free[2]
constexpr int OFF_BAR = OFF_RSTD + 8 * 4;
constexpr int OFF_MISC = OFF_BAR + N_BARS * 8;               // queue[QDEPTH], q_head, dead flag
constexpr int OFF_FINP = OFF_MISC + 256;                     // the finishers' copy of the phase parameters
constexpr int FINP_BYTES = 256;
static_assert(sizeof(SmallMParams) <= FINP_BYTES, "phase parameter copy too small");
static_assert((3 * QDEPTH + 2) * 4 <= 256, "queue area too small");
constexpr int OFF_AUX = OFF_FINP + FINP_BYTES;
constexpr int AUX_PS = 4 * 8 * 16 * 4;
constexpr int AUX_RED = 4 * 2 * 128 * 4;   // [4 warps][2 heads][128] floats per merge round; the merge step reuses it for its weights
static_assert(AUX_RED >= kMaxSplits * 4, "merge weights do not fit");
constexpr int AUX_MLS = 4 * 8 * 2 * 4;
constexpr int AUX_MISC = 128;  // prefix of live splits [9], merge reductions [8], lengths [8]
constexpr int SMEM = OFF_AUX + AUX_PS + AUX_RED + AUX_MLS + AUX_MISC + 128;
static_assert(SMEM <= 227 * 1024, "shared memory budget");

// registers per thread after the warpgroups have traded (launch allocation: 128 each)
constexpr int REGS_WG0 = 72, REGS_CONS = 176, REGS_STAGE = 120, REGS_AUX = 144;
static_assert(REGS_WG0 + REGS_CONS + REGS_STAGE + REGS_AUX <= 4 * 128, "register pool exceeded");

struct F8 {
  float4 a, b;
};

// Moves this warpgroup's per-thread register allocation from the launch value (128) to N: a release
// when N is smaller, a (blocking) request when it is larger.  Every warpgroup calls it exactly once,
// unconditionally, and the four targets add up to the launch total, so the requests are always met.
constexpr int kLaunchRegs = 128;
template <int N>
__device__ __forceinline__ void reg_set() {
  static_assert(N % 8 == 0 && N >= 24 && N <= 256, "register count out of range");
  if constexpr (N > kLaunchRegs) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
  else if constexpr (N < kLaunchRegs) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}

__device__ __forceinline__ int ld_acquire(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_add(int32_t* p, int v) {
  asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ bool aborted(const int32_t* status) {
  return (*reinterpret_cast<const volatile int32_t*>(status) & LADDER_DEV_TIMEOUT) != 0;
}
__device__ __forceinline__ void bar_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
// barrier among `count` threads that also ANDs a predicate: every participant gets the same answer,
// so the decision to leave a role after a failed wait is taken by all its threads together
__device__ __forceinline__ bool bar_and(int id, int count, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 p, %1, 0;\n\t"
      "bar.red.and.pred q, %2, %3, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r)
      : "r"(static_cast<uint32_t>(pred)), "r"(id), "r"(count)
      : "memory");
  return r != 0;
}

// ---- bounded waits; all give up early when another CTA has reported a timeout
// SLEEP_NS > 0: back off between polls.  Used where a few hundred nanoseconds of wake-up latency do not
// matter (finishers, stagers): a waiting warp that keeps polling executes instructions, and at this
// kernel's power draw every instruction costs SM clock.  The back-off times were swept: 2.5 x longer than the first
// choice (1000 / 500 ns at the barriers, 300 / 160 ns at the counters) is faster at every shape (70B 0.25 %, 1.2B
// 1.2 %, parallel layers at the TP-rank slice 1-3 %); 5 x is faster still at the 70B shape (0.7 %) and slower at the
// small ones.
template <int SLEEP_NS = 0>
__device__ __forceinline__ bool wait_mbar(uint64_t* bar, uint32_t parity, const int32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t i = 1;; ++i) {
    if (SLEEP_NS > 0) __nanosleep(SLEEP_NS);
    if (mbar_try_wait_suspend(bar, parity, 4000u)) return true;
    if ((i & 15u) == 0 && (aborted(status) || clock64() - t0 > kWaitCycles)) return false;
  }
}
__device__ __forceinline__ bool wait_counter_gt(const volatile int* ctr, int n, const int32_t* status) {
  if (*ctr > n) return true;
  const long long t0 = clock64();
  for (uint32_t i = 1;; ++i) {
    __nanosleep(160);  // a hot spin would take issue slots from the consumer warp of the same sub-partition
    if (*ctr > n) return true;
    if ((i & 255u) == 0 && (aborted(status) || clock64() - t0 > kWaitCycles)) return false;
  }
}
__device__ __forceinline__ bool wait_global_ge(const int32_t* ctr, int need, const int32_t* status) {
  if (ld_acquire(ctr) >= need) return true;
  const long long t0 = clock64();
  for (uint32_t i = 1;; ++i) {
    __nanosleep(300);
    if (ld_acquire(ctr) >= need) return true;
    if ((i & 31u) == 0 && (aborted(status) || clock64() - t0 > kWaitCycles)) return false;
  }
}
// lane i of the calling warp polls dependency i; the warp agrees on the outcome
__device__ __forceinline__ bool wait_deps(const int* dep, const int* need, int n, const int32_t* counters,
                                          const int32_t* status, int lane) {
  bool ok = true;
  if (lane < n) ok = wait_global_ge(counters + __ldg(dep + lane), __ldg(need + lane), status);
  return __all_sync(0xffffffffu, ok);
}

#define TR_DECL(n)
#define TR_T0()
#define TR_ADD(n)
#define TR_OUT(i, n)

template <typename T>
__device__ __forceinline__ T* ldg_ptr(T* const* p) {  // read-only load of a pointer field
  return reinterpret_cast<T*>(__ldg(reinterpret_cast<const unsigned long long*>(p)));
}

// queue item: phase (10 bits) | first unit (17 bits) | units (4 bits)
__device__ __forceinline__ int item_pack(int ph, int u0, int nu) { return (ph << 21) | (u0 << 4) | nu; }

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

// ------------------------------------------------------------------------------------ attention units
// One split unit: 64 keys x GT query heads sharing a kv head x one sequence, 4 warps (16 keys each).
// Same arithmetic as decode_attention_kernel; loads go through L2 because q and the newest key/value
// row were written by other SMs earlier in this launch.
template <int GT, int DH>
__device__ __forceinline__ void attn_split_unit(const float* q, const kv_t* Kc, const kv_t* Vc,
                                                int n_q_heads, int n_kv_heads, int max_seq_len, int stride_splits,
                                                float* scratch, int b, int split, int hg, int L, float* ps_, float* red_,
                                                float* mls_, int at) {
  constexpr int DPL = DH / 32;
  constexpr int KJ = DH / 32;
  const int warp = at >> 5, lane = at & 31;
  const int g = lane >> 2, tig = lane & 3;
  const int head0 = hg * GT;
  const int group = n_q_heads / n_kv_heads;
  const int kvh = head0 / group;
  const size_t kv_base = (static_cast<size_t>(b) * n_kv_heads + kvh) * max_seq_len * DH;
  const kv_t* K = Kc + kv_base;
  const kv_t* V = Vc + kv_base;
  const int kw0 = split * kChunk + warp * 16;
  const float scale = rsqrtf(static_cast<float>(DH));
  float* ps = ps_ + warp * GT * 16;     // [GT][16]
  float* red = red_;                    // [4][HR][DH], HR heads per merge round
  float* mls = mls_;                    // [4][GT][2]

  uint4 kf[2][KJ];
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
    const int key = kw0 + nt * 8 + g;
#pragma unroll
    for (int j = 0; j < KJ; ++j)
      kf[nt][j] = key < L ? __ldcg(reinterpret_cast<const uint4*>(K + static_cast<size_t>(key) * DH + j * 32 + tig * 8))
                          : make_uint4(0, 0, 0, 0);
  }
  uint32_t vr[16][DPL / 2];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const int key = kw0 + i;
    if (DPL == 4) {
      const uint2 u = key < L ? __ldcg(reinterpret_cast<const uint2*>(V + static_cast<size_t>(key) * DH + lane * DPL))
                              : make_uint2(0, 0);
      vr[i][0] = u.x;
      vr[i][DPL / 2 - 1] = u.y;
    } else {
      vr[i][0] = key < L ? __ldcg(reinterpret_cast<const unsigned int*>(V + static_cast<size_t>(key) * DH + lane * DPL))
                         : 0u;
    }
  }
  uint32_t qa[KJ][2][2], ql[KJ][2][2];
#pragma unroll
  for (int j = 0; j < KJ; ++j)
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float4 v = make_float4(0, 0, 0, 0);
      if (g < GT)
        v = __ldcg(reinterpret_cast<const float4*>(q + (static_cast<size_t>(b) * n_q_heads + head0 + g) * DH + j * 32 +
                                                   tig * 8 + h * 4));
      qa[j][h][0] = pack_f16x2(v.x, v.y);
      qa[j][h][1] = pack_f16x2(v.z, v.w);
      ql[j][h][0] = pack_f16x2(v.x - f16_lo(qa[j][h][0]), v.y - f16_hi(qa[j][h][0]));
      ql[j][h][1] = pack_f16x2(v.z - f16_lo(qa[j][h][1]), v.w - f16_hi(qa[j][h][1]));
    }

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
    *reinterpret_cast<float2*>(&ps[g * 16 + 2 * tig]) = make_float2(sv[0], sv[1]);
    *reinterpret_cast<float2*>(&ps[g * 16 + 8 + 2 * tig]) = make_float2(sv[2], sv[3]);
    if (tig == 0) {
      mls[(warp * GT + g) * 2 + 0] = m;
      mls[(warp * GT + g) * 2 + 1] = l;
    }
  }
  __syncwarp();

  float acc[GT][DPL];
#pragma unroll
  for (int h = 0; h < GT; ++h)
#pragma unroll
    for (int d = 0; d < DPL; ++d) acc[h][d] = 0.f;
#pragma unroll
  for (int i4 = 0; i4 < 4; ++i4) {
    float4 pw[GT];
#pragma unroll
    for (int h = 0; h < GT; ++h) pw[h] = *reinterpret_cast<const float4*>(&ps[h * 16 + i4 * 4]);
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
  // merge the 4 warps and write the unit's partial, HR heads at a time: the staging array holds only
  // [4 warps][HR heads][DH] floats (shared memory is needed for the weight ring)
  constexpr int HR = GT >= 4 ? GT / 4 : 1;
  const int stride = DH + 2;
#pragma unroll
  for (int h0 = 0; h0 < GT; h0 += HR) {
#pragma unroll
    for (int hh = 0; hh < HR; ++hh)
#pragma unroll
      for (int d = 0; d < DPL; ++d) red[(warp * HR + hh) * DH + lane * DPL + d] = acc[h0 + hh][d];
    bar_sync(3, kAux);
    for (int idx = at; idx < HR * DH; idx += kAux) {
      const int hh = idx / DH, h = h0 + hh, d = idx % DH;
      const float m0 = mls[(0 * GT + h) * 2], m1 = mls[(1 * GT + h) * 2], m2 = mls[(2 * GT + h) * 2],
                  m3 = mls[(3 * GT + h) * 2];
      const float M = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
      float o = 0.f, ls = 0.f;
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const float mw = mls[(w * GT + h) * 2];
        const float f = (mw == -INFINITY) ? 0.f : __expf(mw - M);
        o += f * red[(w * HR + hh) * DH + d];
        ls += f * mls[(w * GT + h) * 2 + 1];
      }
      float* dst = scratch + ((static_cast<size_t>(b) * n_q_heads + head0 + h) * stride_splits + split) * stride;
      dst[d] = o;
      if (d == 0) {
        dst[DH] = M;
        dst[DH + 1] = ls;
      }
    }
    bar_sync(3, kAux);  // the staging array (and, after the last round, ps / mls) is rewritten next
  }
}

// Merge of the live splits of one (sequence, head), in split order (same summation order as
// decode_attention_merge_kernel).
template <int DH>
__device__ __forceinline__ void attn_merge_unit(const float* scratch, int n_q_heads, int stride_splits, int n_splits,
                                                int b, int h, float* o, __nv_bfloat16* o_pack, float* wgt, float* red_m,
                                                float* red_l, int at) {
  constexpr int stride = DH + 2;
  const int warp = at >> 5, lane = at & 31;
  const float* base = scratch + (static_cast<size_t>(b) * n_q_heads + h) * stride_splits * stride;
  const bool act = at < DH;
  float m = -INFINITY;
  if (act)
    for (int s = at; s < n_splits; s += DH) {
      wgt[s] = __ldcg(base + s * stride + DH);
      m = fmaxf(m, wgt[s]);
    }
  m = warp_max(m);
  if (lane == 0) red_m[warp] = m;
  bar_sync(3, kAux);
  float M = red_m[0];
#pragma unroll
  for (int w = 1; w < DH / 32; ++w) M = fmaxf(M, red_m[w]);
  float l = 0.f;
  if (act)
    for (int s = at; s < n_splits; s += DH) {
      const float f = (wgt[s] == -INFINITY) ? 0.f : __expf(wgt[s] - M);
      wgt[s] = f;
      l += f * __ldcg(base + s * stride + DH + 1);
    }
  l = warp_sum(l);
  if (lane == 0) red_l[warp] = l;
  bar_sync(3, kAux);
  float lsum = 0.f;
#pragma unroll
  for (int w = 0; w < DH / 32; ++w) lsum += red_l[w];
  if (act) {
    float acc = 0.f;
#pragma unroll 8
    for (int s = 0; s < n_splits; ++s) acc += wgt[s] * __ldcg(base + s * stride + at);
    const float val = lsum > 0.f ? acc / lsum : 0.f;
    o[(static_cast<size_t>(b) * n_q_heads + h) * DH + at] = val;
    if (o_pack) store_packed(o_pack, nullptr, b, h * DH + at, val);  // the output projection's MMA operand
  }
  bar_sync(3, kAux);
}

template <int DH>
__device__ __forceinline__ void attn_split_dispatch(int gt, const float* q, const kv_t* Kc,
                                                    const kv_t* Vc, int n_q_heads, int n_kv_heads,
                                                    int max_seq_len, int stride_splits, float* scratch, int b, int split,
                                                    int hg, int L, float* ps, float* red, float* mls, int at) {
  switch (gt) {
    case 8:
      attn_split_unit<8, DH>(q, Kc, Vc, n_q_heads, n_kv_heads, max_seq_len, stride_splits, scratch, b, split, hg, L, ps,
                             red, mls, at);
      break;
    case 4:
      attn_split_unit<4, DH>(q, Kc, Vc, n_q_heads, n_kv_heads, max_seq_len, stride_splits, scratch, b, split, hg, L, ps,
                             red, mls, at);
      break;
    case 2:
      attn_split_unit<2, DH>(q, Kc, Vc, n_q_heads, n_kv_heads, max_seq_len, stride_splits, scratch, b, split, hg, L, ps,
                             red, mls, at);
      break;
    default:
      attn_split_unit<1, DH>(q, Kc, Vc, n_q_heads, n_kv_heads, max_seq_len, stride_splits, scratch, b, split, hg, L, ps,
                             red, mls, at);
      break;
  }
}

// ------------------------------------------------------------------------------------ the kernel
template <bool PACKED>
__global__ void __launch_bounds__(kThreads, 1) decode_stack_kernel(const StackParams sp) {
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
  uint64_t* norm_ready = act_full + 1;        // [NORM_RING] stagers -> finishers
  uint64_t* red_full = norm_ready + NORM_RING;  // [2] consumers -> finishers
  uint64_t* red_free = red_full + 2;            // [2] finishers -> consumers
  int* queue = reinterpret_cast<int*>(smem + OFF_MISC);  // [QDEPTH] items, then K and chunk count of each item's phase
  volatile int* queue_k = queue + QDEPTH;
  volatile int* queue_nc = queue + 2 * QDEPTH;
  volatile int* q_head = queue + 3 * QDEPTH;
  int* flag_s = queue + 3 * QDEPTH + 1;
  SmallMParams* finp = reinterpret_cast<SmallMParams*>(smem + OFF_FINP);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int batch = sp.batch;
  const int32_t* status = sp.status;

  if (tid == 0) {
    *flag_s = aborted(status) ? 1 : 0;
    *q_head = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 4);
    }
    mbar_init(act_free, 4);
    mbar_init(act_full, 4);
    for (int s = 0; s < NORM_RING; ++s) mbar_init(&norm_ready[s], 4);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&red_full[s], 4);
      mbar_init(&red_free[s], 3);
    }
    fence_barrier_init();
  }
  __syncthreads();
  if (*flag_s) return;  // an earlier launch reported a protocol error: do nothing

  if (warp < 4) {
    reg_set<REGS_WG0>();
    if (warp == 0) {
      // ---------------------------------------------------------------- producer
      const uint64_t pol = l2_policy_evict_first();
      bool ok = true;
      int it = 0, n = 0;
      TR_DECL(ring);
      TR_DECL(claim);
      TR_DECL(total);
      // Which batch comes next is settled one batch ahead of the weight stream, right after the first
      // tile of the current batch has been issued, so the stagers and finishers know early and no
      // round trip of an atomic is exposed.  Whole rounds of a phase's schedule are dealt out
      // statically (claim i to CTA i mod grid): a phase in which every CTA has exactly one batch must
      // not let an early CTA take a second one.  Only the short batches at the end of a long phase are
      // claimed through the counter, which is what evens out the SMs' different streaming rates.
      // The first 128 bytes of a phase descriptor are held across the warp, lane i owning word i, and
      // read with shuffles; the descriptor of the following phase is loaded one phase ahead.
      constexpr int H_W = 0, H_K = 2, H_UNITS = 3, H_NCHUNK = 4, H_WORK = 5, H_STATIC = 7, H_CLAIMS = 8, H_ROUNDS = 9,
                    H_COUNT = 10, H_SIZE = 20;
      static_assert(offsetof(StackPhase, n_static) == 4 * H_STATIC && offsetof(StackPhase, count) == 4 * H_COUNT &&
                        offsetof(StackPhase, size) == 4 * H_SIZE && offsetof(StackPhase, K) == 4 * H_K,
                    "descriptor layout");
      auto load_hdr = [&](int ph) -> int {
        return ph < sp.n_phases ? __ldg(reinterpret_cast<const int*>(sp.phases + ph) + lane) : 0;
      };
      auto H = [&](int h, int idx) -> int { return __shfl_sync(0xffffffffu, h, idx); };
      int cl_ph = 0;    // phase of the next claim
      int cl_k = 0;     // static claims of that phase this CTA has taken
      int cl_pend = 0;  // claim index asked for in phase cl_ph (valid in lane 0)
      int hdr = load_hdr(0), hdr_nx = load_hdr(1);
      // what the item returned by claim_finish belongs to
      const uint8_t* nx_W = nullptr;
      int nx_K = 0, nx_nchunk = 0;
      // ask for the next claim of phase cl_ph (an atomic only for the dynamic tail; its answer is not
      // needed before claim_finish)
      auto claim_issue = [&]() {
        const int n_static = H(hdr, H_STATIC), n_claims = H(hdr, H_CLAIMS), work = H(hdr, H_WORK);
        const int ci = blockIdx.x + cl_k * static_cast<int>(gridDim.x);
        if (ci < n_static) {
          ++cl_k;
          cl_pend = ci;
        } else if (n_static < n_claims) {
          if (lane == 0) cl_pend = n_static + atomicAdd(sp.counters + work, 1);
        } else {
          cl_pend = n_claims;
        }
      };
      // turn the claim into the next item (moving on to later phases while a phase has nothing left
      // for this CTA), publish it; 0 = end of the step
      auto claim_finish = [&]() -> int {
        int item = 0;
        for (;;) {
          int ci = __shfl_sync(0xffffffffu, cl_pend, 0), u0 = 0, nu = 0;
          if (ci < H(hdr, H_CLAIMS)) {
            int ubase = 0;
            const int sn = H(hdr, H_ROUNDS), n_units = H(hdr, H_UNITS);
            for (int r = 0; r < sn; ++r) {
              const int cnt = H(hdr, H_COUNT + r), sz = H(hdr, H_SIZE + r);
              if (ci < cnt) {
                u0 = ubase + ci * sz;
                nu = min(sz, n_units - u0);
                break;
              }
              ci -= cnt;
              ubase += cnt * sz;
            }
          }
          if (nu > 0) {
            item = item_pack(cl_ph, u0, nu) | (1 << 31);
            nx_K = H(hdr, H_K);
            nx_nchunk = H(hdr, H_NCHUNK);
            nx_W = reinterpret_cast<const uint8_t*>(
                (static_cast<unsigned long long>(static_cast<unsigned int>(H(hdr, H_W + 1))) << 32) |
                static_cast<unsigned int>(H(hdr, H_W)));
            break;
          }
          ++cl_ph;  // nothing left for this CTA in this phase
          cl_k = 0;
          if (cl_ph >= sp.n_phases) break;
          hdr = hdr_nx;
          hdr_nx = load_hdr(cl_ph + 1);
          claim_issue();
        }
        if (lane == 0) {
          queue[n % QDEPTH] = item ? (item & 0x7fffffff) : -1;
          queue_k[n % QDEPTH] = nx_K;
          queue_nc[n % QDEPTH] = nx_nchunk;
          __threadfence_block();
          *q_head = n + 1;
        }
        ++n;
        return item;
      };
      int item;
      {
        TR_T0();
        claim_issue();
        item = claim_finish();
        TR_ADD(claim);
      }
      while (ok && item != 0) {
        const int u0 = (item >> 4) & 0x1ffff, nu = item & 15;
        const uint8_t* Wb = nx_W;
        const int K = nx_K, nchunk = nx_nchunk;
        {  // ask for the batch after this one; the answer is picked up two tiles later
          TR_T0();
          claim_issue();
          TR_ADD(claim);
        }
        const int resolve_at = min(2, nchunk * nu - 1);
        int issued = 0;
        int next_item = 0;
        const int row0 = u0 * 8;
        for (int ch = 0; ch < nchunk && ok; ++ch) {
          const int k0 = ch * TK;
          const uint32_t kb = static_cast<uint32_t>(min(TK, K - k0)) * 2u;
          for (int h8 = 0; h8 < nu; ++h8) {
            const int st = it % STAGES;
            {
              TR_T0();
              ok = __all_sync(0xffffffffu, wait_mbar(&empty[st], ((it / STAGES) & 1) ^ 1u, status));
              TR_ADD(ring);
            }
            if (!ok) break;
            if (lane == 0) mbar_expect_tx(&full[st], 8 * kb);
            __syncwarp();
            if (lane < 8) {
              const size_t row = static_cast<size_t>(row0 + h8 * 8 + lane);
              bulk_g2s(ring + st * STAGE_BYTES + lane * PITCH, Wb + (row * K + k0) * 2, kb, &full[st], pol);
            }
            ++it;
            if (issued++ == resolve_at) {  // tiles are on their way: publish what comes next
              TR_T0();
              next_item = claim_finish();
              TR_ADD(claim);
            }
          }
        }
        item = next_item;
      }
      if (!ok && lane == 0) {  // protocol error: release the other roles
        queue[n % QDEPTH] = -1;
        __threadfence_block();
        *q_head = n + 1;
      }
      if (!ok && lane == 0) atomicOr(sp.status, LADDER_DEV_TIMEOUT);
      if (!ok) {  // wait (bounded) for the copies in flight before the CTA may exit
        for (int j = 1; j <= STAGES && j <= it; ++j) {
          const int i2 = it - j;
          mbar_wait_bounded(&full[i2 % STAGES], (i2 / STAGES) & 1);
        }
      }
      return;
    }

    // ------------------------------------------------------------------ finishers (warps 1-3)
    const int ft = tid - 32;  // 0..95
    bool ok = true;
    int cur_ph = -1, norm_cnt = 0;
    bool phase_norm = false, have_rstd = true;
    int32_t* done_ctr = nullptr;
    TR_DECL(fdeps);
    TR_DECL(fred);
    TR_DECL(fq);
    TR_DECL(ftotal);
    for (int n = 0;; ++n) {
      {
        TR_T0();
        ok = bar_and(2, kFin, ok && wait_counter_gt(q_head, n, status));
        TR_ADD(fq);
      }
      if (!ok) break;
      const int id = reinterpret_cast<volatile int*>(queue)[n % QDEPTH];
      if (id < 0) break;
      const int ph = id >> 21, row0 = ((id >> 4) & 0x1ffff) * 8, nu = id & 15, rows = nu * 8;
      if (ph != cur_ph) {
        const StackPhase* P = sp.phases + ph;
        // private copy of the phase's epilogue description
        const int* src = reinterpret_cast<const int*>(&P->p);
        int* dst = reinterpret_cast<int*>(finp);
        for (int i = ft; i < static_cast<int>(sizeof(SmallMParams) / 4); i += kFin) dst[i] = __ldg(src + i);
        phase_norm = __ldg(&P->act_mode) == ACT_F32_NORM;
        have_rstd = !phase_norm;
        done_ctr = sp.counters + __ldg(&P->done_idx);
        // what the epilogue reads (addend) must be written, what it overwrites must have been read
        {
          TR_T0();
          ok = bar_and(2, kFin, wait_deps(P->epi_dep, P->epi_need, P->n_epi_deps, sp.counters, status, lane));
          TR_ADD(fdeps);
        }
        if (!ok) break;
        cur_ph = ph;
      }
      const int slot = n & 1;
      {
        TR_T0();
        bool okw = wait_mbar<1000>(&red_full[slot], (n >> 1) & 1, status);
        if (!have_rstd)
          okw = okw && wait_mbar<1000>(&norm_ready[norm_cnt & (NORM_RING - 1)], (norm_cnt / NORM_RING) & 1, status);
        ok = bar_and(2, kFin, okw);
        TR_ADD(fred);
      }
      if (!ok) break;
      if (!have_rstd) {  // 1/rms of every activation row, once per phase and CTA
        if (ft < batch) {
          const float* sq = ssq_part + (norm_cnt & (NORM_RING - 1)) * 32;
          const float s = sq[ft] + sq[8 + ft] + sq[16 + ft] + sq[24 + ft];
          rstd_s[ft] = rsqrtf(s / static_cast<float>(finp->K) + finp->eps);
        }
        bar_sync(2, kFin);
        have_rstd = true;
        ++norm_cnt;
      }
      const float* rs = red + slot * RED_FLOATS;
      auto column = [&](int a, int rr, int c) -> float {
        const int idx = (a * 4 + ((rr >> 3) * 2 + (c & 1))) * 32 + ((rr & 7) * 4 + (c >> 1));
        return rs[idx] + rs[RG_MAX * 128 + idx] + rs[2 * RG_MAX * 128 + idx] + rs[3 * RG_MAX * 128 + idx];
      };
      auto value = [&](int r, int b) -> float {
        const int a = r >> 4, rr = r & 15;
        float s = column(a, rr, b);
        if (PACKED) s += column(a, rr, b + 4);  // high-part product + low-part product
        if (phase_norm) s *= rstd_s[b];
        return s;
      };
      smallm_epilogue<kFin>(*finp, ft, rows, row0, batch, value);
      // all finisher threads' outputs are ordered before the release by the barrier (the release is cumulative)
      bar_sync(2, kFin);
      if (ft == 0) red_release_add(done_ctr, nu);
      if (lane == 0) mbar_arrive(&red_free[slot]);
    }
    if (!ok && lane == 0) atomicOr(sp.status, LADDER_DEV_TIMEOUT);
    return;
  }

  if (warp < 8) {
    // -------------------------------------------------------------------- consumers (warps 4-7)
    reg_set<REGS_CONS>();
    const int cw = warp - 4;
    const int g = lane >> 2, tig = lane & 3;
    const uint32_t ring_u32 = smem_u32(ring);
    const uint32_t act_u32 = smem_u32(act);
    // which activation row feeds MMA column g: packed = hi rows 0-3 then lo rows 4-7 of batch g & 3
    const bool col_valid = PACKED ? ((g & 3) < batch) : (g < batch);
    bool ok = true;
    uint4 bf[SPW];
#pragma unroll
    for (int j = 0; j < SPW; ++j) bf[j] = make_uint4(0, 0, 0, 0);
    int it = 0, n_req = 0, cur_ph = -1, K = 0, nchunk = 0;
    TR_DECL(cq);
    TR_DECL(cact);
    TR_DECL(cw);
    TR_DECL(cred);
    TR_DECL(cmma);
    TR_DECL(ctotal);
    for (int n = 0;; ++n) {
      {
        TR_T0();
        ok = __all_sync(0xffffffffu, ok && wait_counter_gt(q_head, n, status));
        TR_ADD(cq);
      }
      if (!ok) break;
      const int id = reinterpret_cast<volatile int*>(queue)[n % QDEPTH];
      if (id < 0) break;
      const int ph = id >> 21;
      if (ph != cur_ph) {
        K = queue_k[n % QDEPTH];
        nchunk = queue_nc[n % QDEPTH];
        cur_ph = ph;
      }
      const int rows = (id & 15) * 8;
      const int rgn = (rows + 15) >> 4;

      float acc[RG_MAX][2][4];
#pragma unroll
      for (int a = 0; a < RG_MAX; ++a)
#pragma unroll
        for (int q = 0; q < 2; ++q)
#pragma unroll
          for (int c = 0; c < 4; ++c) acc[a][q][c] = 0.f;

      for (int ch = 0; ch < nchunk && ok; ++ch) {
        const int k0 = ch * TK;
        // hoist this warp's activation fragments of the chunk, then hand the buffer back
        {
          TR_T0();
          ok = __all_sync(0xffffffffu, wait_mbar(act_full, n_req & 1, status));
          TR_ADD(cact);
        }
        if (!ok) break;
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
          if (rgi >= rgn || !ok) break;  // uniform across the warp
          const bool hi_valid = (rgi * 16 + 8) < rows;
          const int st0 = it % STAGES, st1 = (it + 1) % STAGES;
          {
            TR_T0();
            bool okw = wait_mbar(&full[st0], (it / STAGES) & 1, status);
            if (okw && hi_valid) okw = wait_mbar(&full[st1], ((it + 1) / STAGES) & 1, status);
            ok = __all_sync(0xffffffffu, okw);
            TR_ADD(cw);
          }
          if (!ok) break;
          const uint32_t base0 = ring_u32 + st0 * STAGE_BYTES + g * PITCH + tig * 16;
          const uint32_t base1 = ring_u32 + st1 * STAGE_BYTES + g * PITCH + tig * 16;
          // a full chunk with both 8-row halves present (the common case) takes the path without
          // predicates: a guarded shared-memory load compiles to a branch, and 64 of them per tile
          // cost more than the loads and MMAs themselves
          if (hi_valid && k0 + TK <= K) slab_loop<true>(acc[rgi][0], acc[rgi][1], bf, base0, base1, cw, k0, K, tig, true);
          else slab_loop<false>(acc[rgi][0], acc[rgi][1], bf, base0, base1, cw, k0, K, tig, hi_valid);
          __syncwarp();
          if (lane == 0) {
            mbar_arrive(&empty[st0]);
            if (hi_valid) mbar_arrive(&empty[st1]);
          }
          it += hi_valid ? 2 : 1;
        }
      }
      if (!ok) break;

      // hand the accumulator fragments to the finishers and move on
      const int slot = n & 1;
      {
        TR_T0();
        ok = __all_sync(0xffffffffu, wait_mbar(&red_free[slot], ((n >> 1) & 1) ^ 1u, status));
        TR_ADD(cred);
      }
      if (!ok) break;
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
    if (!ok && lane == 0) atomicOr(sp.status, LADDER_DEV_TIMEOUT);
    return;
  }

  if (warp < 12) {
    // -------------------------------------------------------------------- stagers (warps 8-11)
    reg_set<REGS_STAGE>();
    const int st = tid - 256;  // 0..127
    const int sw = warp - 8;
    const uint32_t act_u32 = smem_u32(act);
    bool ok = true;
    int cur_ph = -1, K = 0, nchunk = 0, norm_cnt = 0, r = 0;
    bool norm = false, ssq_on = false;
    const float* actf = nullptr;
    const __nv_bfloat16* gain = nullptr;
    static_assert(offsetof(StackPhase, act) == 128 && offsetof(StackPhase, gain) == 136 &&
                      offsetof(StackPhase, act_mode) == 144 && offsetof(StackPhase, n_act_deps) == 148 &&
                      offsetof(StackPhase, act_dep) == 152 && offsetof(StackPhase, act_need) == 152 + 4 * kStackMaxDeps &&
                      offsetof(StackPhase, act_packed) == 128 + 4 * 28,
                  "descriptor layout");
    auto load_h1 = [&](int ph) -> int {
      return ph < sp.n_phases ? __ldg(reinterpret_cast<const int*>(sp.phases + ph) + 32 + lane) : 0;
    };
    int h1_nx_ph = 0, h1_nx = load_h1(0);
    float ssq[8];
#pragma unroll
    for (int b = 0; b < 8; ++b) ssq[b] = 0.f;

    constexpr int SU = TK / 1024;  // 1024-element sub-blocks per chunk (128 threads x 8 elements each)
    F8 x[4][SU];
    uint4 gq[SU];
    bool kv[SU];
    auto load_rows = [&](int ch, int round) {
      const int k0 = ch * TK;
#pragma unroll
      for (int u = 0; u < SU; ++u) {
        const int k = k0 + (st + u * 128) * 8;
        kv[u] = k < K;
        gq[u] = make_uint4(0x3f803f80u, 0x3f803f80u, 0x3f803f80u, 0x3f803f80u);  // gain 1.0
        if (norm) gq[u] = kv[u] ? __ldcg(reinterpret_cast<const uint4*>(gain + k)) : make_uint4(0, 0, 0, 0);  // L2: keeps L1 for the descriptors
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int u = 0; u < SU; ++u) {
          const int b = round * 4 + i;
          x[i][u].a = x[i][u].b = make_float4(0, 0, 0, 0);
          if (kv[u] && b < batch) {
            const float4* src =
                reinterpret_cast<const float4*>(actf + static_cast<size_t>(b) * K + k0 + (st + u * 128) * 8);
            x[i][u].a = __ldcg(src);
            x[i][u].b = __ldcg(src + 1);
          }
        }
    };
    auto store_rows = [&](int round) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int b = round * 4 + i;
        if (b >= batch) break;
#pragma unroll
        for (int u = 0; u < SU; ++u) {
          float y[8] = {x[i][u].a.x, x[i][u].a.y, x[i][u].a.z, x[i][u].a.w,
                        x[i][u].b.x, x[i][u].b.y, x[i][u].b.z, x[i][u].b.w};
          if (norm) {
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
          if (PACKED) {
            uint4 lo;
            lo.x = pack_bf16x2(y[0] - bf16_lo(hi.x), y[1] - bf16_hi(hi.x));
            lo.y = pack_bf16x2(y[2] - bf16_lo(hi.y), y[3] - bf16_hi(hi.y));
            lo.z = pack_bf16x2(y[4] - bf16_lo(hi.z), y[5] - bf16_hi(hi.z));
            lo.w = pack_bf16x2(y[6] - bf16_lo(hi.w), y[7] - bf16_hi(hi.w));
            sts128(dst + 4 * PITCH, lo);
          }
        }
      }
    };

    auto sumsq_rows = [&]() {  // the sums of squares exactly as store_rows forms them, nothing else
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (i >= batch) break;
#pragma unroll
        for (int u = 0; u < SU; ++u) {
          const float y[8] = {x[i][u].a.x, x[i][u].a.y, x[i][u].a.z, x[i][u].a.w,
                              x[i][u].b.x, x[i][u].b.y, x[i][u].b.z, x[i][u].b.w};
          ssq[i] += y[0] * y[0] + y[1] * y[1] + y[2] * y[2] + y[3] * y[3] + y[4] * y[4] + y[5] * y[5] +
                    y[6] * y[6] + y[7] * y[7];
        }
      }
    };
    const __nv_bfloat16* actp = nullptr;
    TR_DECL(sdeps);
    TR_DECL(sfree);
    TR_DECL(sq);
    TR_DECL(stotal);
    for (int n = 0;; ++n) {
      {
        TR_T0();
        ok = __all_sync(0xffffffffu, ok && wait_counter_gt(q_head, n, status));
        TR_ADD(sq);
      }
      if (!ok) break;
      const int id = reinterpret_cast<volatile int*>(queue)[n % QDEPTH];
      if (id < 0) break;
      const int ph = id >> 21;
      if (ph != cur_ph) {
        // second 128 bytes of the descriptor, lane i owning word i; the next phase's were loaded ahead
        const int h1 = (ph == h1_nx_ph) ? h1_nx : load_h1(ph);
        h1_nx_ph = ph + 1;
        h1_nx = load_h1(ph + 1);
        K = queue_k[n % QDEPTH];
        nchunk = queue_nc[n % QDEPTH];
        actf = reinterpret_cast<const float*>((static_cast<unsigned long long>(static_cast<unsigned int>(
                                                   __shfl_sync(0xffffffffu, h1, 1)))
                                               << 32) |
                                              static_cast<unsigned int>(__shfl_sync(0xffffffffu, h1, 0)));
        gain = reinterpret_cast<const __nv_bfloat16*>(
            (static_cast<unsigned long long>(static_cast<unsigned int>(__shfl_sync(0xffffffffu, h1, 3))) << 32) |
            static_cast<unsigned int>(__shfl_sync(0xffffffffu, h1, 2)));
        norm = __shfl_sync(0xffffffffu, h1, 4) == ACT_F32_NORM;
        actp = reinterpret_cast<const __nv_bfloat16*>(
            (static_cast<unsigned long long>(static_cast<unsigned int>(__shfl_sync(0xffffffffu, h1, 29))) << 32) |
            static_cast<unsigned int>(__shfl_sync(0xffffffffu, h1, 28)));
        ssq_on = norm;  // the first batch of a normalised phase also forms the sums of squares
        cur_ph = ph;
        // the activations of this phase must have been written (all of them: every batch needs all of K)
        {
          TR_T0();
          // lane i polls dependency i (words 6.. = counter index, 6 + kStackMaxDeps.. = required value)
          const int nd = __shfl_sync(0xffffffffu, h1, 5);
          const int dep_i = __shfl_sync(0xffffffffu, h1, 6 + (lane < kStackMaxDeps ? lane : 0));
          const int need_i = __shfl_sync(0xffffffffu, h1, 6 + kStackMaxDeps + (lane < kStackMaxDeps ? lane : 0));
          bool okd = true;
          if (lane < nd) okd = wait_global_ge(sp.counters + dep_i, need_i, status);
          ok = __all_sync(0xffffffffu, okd);
          __syncwarp();
          TR_ADD(sdeps);
        }
        if (!ok) break;
      }
      // chunk by chunk, one chunk ahead of the consumers: the raw values are loaded into registers
      // before the buffer is handed back (act_free)
      for (int ch = 0; ch < nchunk; ++ch, ++r) {
        // Operands already in MMA form (written by the producing phase's epilogue): the chunk is copied as it
        // is with cp.async (16 bytes per copy, L2 -> shared memory, generic proxy: coherent like ld.global.cg)
        // once the buffer has been handed back.  Otherwise convert from fp32.  The fp32 rows are still read
        // while the first batch of a normalised phase is staged, for the sums of squares only.
        const bool copy = actp != nullptr;
        if (copy && ssq_on) {  // the fp32 rows first (their registers are then free for the copy)
          load_rows(ch, 0);
          sumsq_rows();
        }
        if (!copy) load_rows(ch, 0);
        {
          TR_T0();
          ok = __all_sync(0xffffffffu, wait_mbar<500>(act_free, (r & 1) ^ 1u, status));
          TR_ADD(sfree);
        }
        if (!ok) break;
        if (copy) {  // 16 x 16 bytes per thread, global (L2) -> shared memory without a register round trip
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int idx = st + j * 128, row = idx >> 8, col = idx & 255;  // 256 16-byte units per 4 KB row
            const __nv_bfloat16* src = actp + (static_cast<size_t>(ch) * 8 + row) * TK + col * 8;
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(act_u32 + row * PITCH + col * 16), "l"(src)
                         : "memory");
          }
          asm volatile("cp.async.wait_all;" ::: "memory");
        } else {
          store_rows(0);
          if (!PACKED && batch > 4) {
            load_rows(ch, 1);
            store_rows(1);
          }
        }
        if (ssq_on && ch == nchunk - 1) {  // every chunk has been staged once: publish the sums
          float* sq = ssq_part + (norm_cnt & (NORM_RING - 1)) * 32;
#pragma unroll
          for (int b = 0; b < 8; ++b) {
            if (b < batch) {
              const float t = warp_sum(ssq[b]);
              if (lane == 0) sq[sw * 8 + b] = t;
            }
            ssq[b] = 0.f;
          }
          ssq_on = false;
          __syncwarp();
          if (lane == 0) mbar_arrive(&norm_ready[norm_cnt & (NORM_RING - 1)]);
          ++norm_cnt;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(act_full);
      }
      if (!ok) break;
    }
    if (!ok && lane == 0) atomicOr(sp.status, LADDER_DEV_TIMEOUT);
    return;
  }

  // ---------------------------------------------------------------------- attention (warps 12-15)
  reg_set<REGS_AUX>();
  {
    const int at = tid - 384;  // 0..127
    float* ps = reinterpret_cast<float*>(smem + OFF_AUX);
    float* ared = reinterpret_cast<float*>(smem + OFF_AUX + AUX_PS);
    float* mls = reinterpret_cast<float*>(smem + OFF_AUX + AUX_PS + AUX_RED);
    int* pre = reinterpret_cast<int*>(smem + OFF_AUX + AUX_PS + AUX_RED + AUX_MLS);  // [9] prefix of live splits
    float* red_m = reinterpret_cast<float*>(pre + 12);
    float* red_l = red_m + 4;
    int* lens_s = pre + 20;  // [8] keys attended per sequence
    bool ok = true;
    if (sp.n_attn > 0) {
      if (at == 0) {
        const DecodeAttnParams& a0 = sp.attn[0].a;
        int acc = 0;
        pre[0] = 0;
        for (int b = 0; b < batch; ++b) {
          int L = a0.kv_len[b] + a0.kv_len_offset;
          L = max(0, min(L, a0.max_seq_len));
          lens_s[b] = L;
          acc += (L + kChunk - 1) / kChunk;
          pre[b + 1] = acc;
        }
      }
    }
    bar_sync(3, kAux);
    for (int li = 0; li < sp.n_attn; ++li) {
      const StackAttn* A = sp.attn + li;
      const float* q = A->a.q;
      const kv_t* Kc = A->a.k;
      const kv_t* Vc = A->a.v;
      const int Hq = A->a.n_q_heads, Hkv = A->a.n_kv_heads, DH = A->a.head_dim, max_seq = A->a.max_seq_len;
      const int stride_splits = A->a.n_splits;
      float* scratch = A->a.scratch;
      float* o = A->a.o;
      __nv_bfloat16* o_pack = PACKED ? A->o_pack : nullptr;
      int gt = 1;
      {
        const int group = Hq / Hkv;
        while (gt < 8 && group % (gt * 2) == 0) gt *= 2;
      }
      const int HG = Hq / gt;
      // While the QKV phase of this layer is still running: pull the cached keys and values of the layer
      // (everything but this step's row) into L2, so that the split units, which are on the critical path of
      // small models, do not queue behind the weight stream in DRAM.  This CTA's share of the 128-byte lines.
      // Only where the prefix is small (<= 8 MB per layer): at large shapes the gate/up phase hides the attention
      // anyway and the prefetch only competes with the weight stream.
      const size_t row_lines = static_cast<size_t>(DH) * 2 / 128;
      if (static_cast<size_t>(pre[batch]) * kChunk * row_lines * Hkv * 2 * 128 <= (size_t(8) << 20)) {
        for (int b = 0; b < batch; ++b) {
          const int rows = max(0, lens_s[b] - 1);
          const size_t per_head = static_cast<size_t>(rows) * row_lines;
          const size_t total_lines = per_head * Hkv;
          for (size_t i = static_cast<size_t>(blockIdx.x) * kAux + at; i < total_lines;
               i += static_cast<size_t>(gridDim.x) * kAux) {
            const size_t hk = i / per_head, r = i - hk * per_head;
            const size_t off = ((static_cast<size_t>(b) * Hkv + hk) * max_seq) * DH + r * 64;  // bf16 elements
            asm volatile("prefetch.global.L2 [%0];" ::"l"(Kc + off));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(Vc + off));
          }
        }
      }
      // q and this step's key/value rows are written; the partials of the previous layer are merged
      ok = bar_and(3, kAux, wait_deps(A->dep, A->need, A->n_deps, sp.counters, status, lane));
      if (!ok) break;
      const int total = pre[batch] * HG;
      int mine = 0;
      for (int u = blockIdx.x; u < total; u += gridDim.x) {
        const int hg = u % HG, t = u / HG;
        int b = 0;
        while (b + 1 < batch && t >= pre[b + 1]) ++b;
        const int split = t - pre[b];
        const int L = lens_s[b];
        if (DH == 128)
          attn_split_dispatch<128>(gt, q, Kc, Vc, Hq, Hkv, max_seq, stride_splits, scratch, b, split, hg, L, ps, ared,
                                   mls, at);
        else
          attn_split_dispatch<64>(gt, q, Kc, Vc, Hq, Hkv, max_seq, stride_splits, scratch, b, split, hg, L, ps, ared, mls,
                                  at);
        ++mine;
      }
      bar_sync(3, kAux);
      if (at == 0 && mine > 0) red_release_add(sp.counters + A->split_done, mine);
      // all partials of this layer (every CTA's) before any merge; o free to overwrite
      bool okw = true;
      if (lane == 0) okw = wait_global_ge(sp.counters + A->split_done, total, status);
      okw = __all_sync(0xffffffffu, okw) && wait_deps(A->mdep, A->mneed, A->n_mdeps, sp.counters, status, lane);
      ok = bar_and(3, kAux, okw);
      if (!ok) break;
      const int n_pairs = batch * Hq;
      mine = 0;
      for (int u = blockIdx.x; u < n_pairs; u += gridDim.x) {
        const int b = u / Hq, h = u % Hq;
        const int ns = pre[b + 1] - pre[b];
        if (DH == 128) attn_merge_unit<128>(scratch, Hq, stride_splits, ns, b, h, o, o_pack, ared, red_m, red_l, at);
        else attn_merge_unit<64>(scratch, Hq, stride_splits, ns, b, h, o, o_pack, ared, red_m, red_l, at);
        ++mine;
      }
      bar_sync(3, kAux);
      if (at == 0 && mine > 0) red_release_add(sp.counters + A->merge_done, mine);
    }
    if (!ok && lane == 0) atomicOr(sp.status, LADDER_DEV_TIMEOUT);
  }
}

bool g_stack_usable = false;

}  // namespace


cudaError_t decode_stack_init(int sm_count, bool* usable) {
  *usable = false;
  cudaError_t e = cudaFuncSetAttribute(decode_stack_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(decode_stack_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
  if (e != cudaSuccess) return e;
  // The warpgroups trade registers at run time (setmaxnreg); the totals above assume the launch
  // allocation of 128 per thread.  Anything else: do not use the kernel.
  cudaFuncAttributes fa;
  e = cudaFuncGetAttributes(&fa, decode_stack_kernel<true>);
  if (e != cudaSuccess) return e;
  bool ok = fa.numRegs == 128;
  e = cudaFuncGetAttributes(&fa, decode_stack_kernel<false>);
  if (e != cudaSuccess) return e;
  ok = ok && fa.numRegs == 128;
  int dev = 0, coop = 0, per_sm = 0;
  e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
  if (e == cudaSuccess)
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_stack_kernel<true>, kThreads, SMEM);
  if (e != cudaSuccess) return e;
  (void)sm_count;
  g_stack_usable = ok && coop && per_sm >= 1;
  *usable = g_stack_usable;
  return cudaSuccess;
}

cudaError_t launch_decode_stack(const StackParams& sp, int sm_count, cudaStream_t stream) {
  if (!g_stack_usable || sp.batch < 1 || sp.batch > 8 || sp.n_phases > kStackMaxPhases || !sp.status || !sp.counters)
    return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(sm_count);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = SMEM;
  cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeCooperative;  // all CTAs co-resident: they wait on one another's counters
  at[0].val.cooperative = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  // batch <= 4 only: there the bf16 hi and lo parts of the activations share one 8-column MMA tile.  Batches 5..8
  // would have to run with a single bf16 value per activation (measured: 4e-3 hidden-state error at 4 layers against
  // 3e-4 with the pair), so they take the tcgen05 kernels, which carry the pair at any batch.
  if (sp.batch > 4) return cudaErrorInvalidValue;
  return cudaLaunchKernelEx(&cfg, decode_stack_kernel<true>, sp);
}

}  // namespace ladder
