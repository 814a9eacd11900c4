// Grouped-query decode attention for wide batches (batch > 8, head_dim 128) on TMA + tcgen05.
//
// At batch <= 8 the cached prefix is ~1 % of a decode step's bytes and attention is a latency problem
// (decode_attention.cu); at batch 16..64 it is 10-20 % of the bytes and a bandwidth problem, which the register-
// fragment kernel cannot feed (it stops near 3.4 TB/s of keys and values: every byte passes through a load
// instruction, a register and a shuffle or permute of a consumer warp).  Here the TMA unit streams K / V tiles of
// 128 cache rows into a three-slot shared-memory ring and the tensor core reads them from there:
//   work item = (128-key tile, kv head, sequence); persistent CTAs, one per SM, each with a contiguous range of the
//                    live tiles;
//   S^T[key, head] = K_tile[128 keys x 128] . Q^T       tcgen05.mma M 128 (keys), N 16, K 128: the B operand holds the
//                    query heads of the kv group (at most 8) as a binary16 hi part in rows 0-7 and the lo part in rows
//                    8-15, so one round of MMAs gives both partial scores; converted from fp32 by a warp of this
//                    kernel, once per (sequence, kv head) group of a CTA's range and a group ahead;
//   softmax over the tile's keys: a thread owns one key (one TMEM lane), so the per-head maximum and sum are
//                    reductions across the 128 threads (shuffles, then four values per head through shared memory);
//   O^T[dim, head] = V_tile^T[128 dims x 128 keys] . P^T   V straight from the cache layout as an MN-major A operand,
//                    P^T as a binary16 hi + lo pair (rows 0-7 / 8-15 of one B operand) written to shared memory by
//                    the softmax warps;
//   the tile's partial (o, m, l) goes to the scratch the merge kernel of decode_attention.cu reads (one partial per
//                    128 keys instead of per 64); tiles beyond a sequence's length get an empty partial.
// 448 threads: warps 0-3 and 4-7 two softmax warpgroups that take the CTA's items in turn (the per-item chain of
// TMEM load, cross-warp maximum, exp2, cross-warp sum and P store is latency, not work: two in flight hide each
// other), warps 8-11 epilogue, warps 12 / 15 TMA producers of the key / value tiles, warps 13 / 14 MMA issuers of the
// scores / the P.V products, warp 16 query conversion.  Keys and values have rings and issuers of their own on purpose:
// with one producer and one issuer working through "K(n+1), V(n)" and "scores(n+1), P.V(n)" in program order, a
// P.V product that was ready waited behind the scores of a tile still in flight, its slot was released late, and no
// more than about one tile per SM was ever on its way from memory (3.7 TB/s).
// Key rows at or beyond the sequence's length are masked, and their value rows are zeroed in shared memory before
// the MMA reads them (stale cache bytes may be NaN).  Every wait is bounded; a protocol error sets the status word.
#include <cuda.h>

#include "common.cuh"
#include "kernels.h"
#include "tcgen05_attn.cuh"

namespace ladder {
namespace {

constexpr int kDT = 128;          // keys per tile
constexpr int kDThreads = 544;
constexpr int kDH = 128;          // head_dim
constexpr int kNH = 8;            // query heads per kv head at most; the MMAs' N is 2 kNH (hi rows, lo rows)
constexpr int kMaxBatch = 256;    // sequence lengths are held in shared memory
constexpr int KV_TILE = 2 * BLK_BYTES;              // 128 rows x 128 binary16
constexpr int D_SLOTS = 3;
constexpr int Q_TILE = 2 * 16 * 128;                // 16 rows (8 hi, 8 lo) x 128 binary16 as two 64-column blocks of 16 x 128 B
constexpr int OFF_K = 0, OFF_V = D_SLOTS * KV_TILE; // K slots, then V slots
constexpr int OFF_Q = 2 * D_SLOTS * KV_TILE;        // [2 items]
constexpr int OFF_P = OFF_Q + 2 * Q_TILE;           // [2 softmax warpgroups]
constexpr int OFF_STAT = OFF_P + 2 * Q_TILE;        // float red[2 warpgroups][2][4][8] (maxima), float m[4][8], float sums[4][4][8], int lens[256]
constexpr int OFF_DBAR = OFF_STAT + (128 + 32 + 128 + 2 * kMaxBatch + 8) * 4;
constexpr int D_SMEM = OFF_DBAR + 40 * 8 + 1024;
constexpr uint32_t IDESC_S = (1u << 4) | (static_cast<uint32_t>(2 * kNH >> 3) << 17) | (static_cast<uint32_t>(128 >> 4) << 24);
constexpr uint32_t IDESC_O = IDESC_S | (1u << 15);  // A (the value tile) is MN-major
constexpr int D_TMEM_COLS = 64;                     // S^T at 0 / 16, O^T at 32 / 48 (hi columns 0-7, lo columns 8-15 each)

struct DtParams {
  const float* q;          // [batch, Hq*128] fp32
  const int32_t* kv_len;
  int kv_len_offset, batch, n_q_heads, n_kv_heads, max_seq_len;
  int n_tiles;             // tiles per (sequence, kv head) = partials per (sequence, head)
  int n_items;             // batch * n_kv_heads * n_tiles
  float* scratch;          // [batch][Hq][n_tiles][130]
  int32_t* status;
};

// A CTA's work: a contiguous range of the live tiles in (sequence, kv head, tile) order, so that consecutive items
// mostly share their (sequence, kv head) -- one query conversion per group of tiles instead of one per tile, and key /
// value rows that follow one another in memory.  Every role walks the range with its own copy of this cursor.
struct DtItem {
  int b, kvh, tile, L;  // the tile, and the keys its sequence attends
  int ntile;            // live tiles of this sequence
  int left;             // tiles left in the CTA's range, this one included; 0: done
  int g;                // index of the (sequence, kv head) group among those this CTA touches
  bool first;           // first tile of its group within this CTA's range
  __device__ __forceinline__ bool last_of_group() const { return tile + 1 == ntile || left == 1; }
};
__device__ __forceinline__ int dt_tiles(int L) { return (L + kDT - 1) / kDT; }
// pre[b] = live tiles of the sequences before b, times the kv heads (pre[batch] = all live tiles)
__device__ __forceinline__ void dt_begin(const DtParams& p, const int* lens, const int* pre, DtItem& t) {
  const int total = pre[p.batch];
  const int per = (total + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
  const int start = min(total, static_cast<int>(blockIdx.x) * per);
  t.left = min(total, start + per) - start;
  t.g = 0;
  t.first = true;
  t.b = t.kvh = t.tile = t.L = 0;
  t.ntile = 1;
  if (t.left <= 0) return;
  int b = 0;
  while (pre[b + 1] <= start) ++b;
  t.b = b;
  t.L = lens[b];
  t.ntile = dt_tiles(t.L);
  const int r = start - pre[b];
  t.kvh = r / t.ntile;
  t.tile = r - t.kvh * t.ntile;
}
__device__ __forceinline__ void dt_advance(const DtParams& p, const int* lens, DtItem& t) {
  if (--t.left <= 0) return;
  t.first = false;
  if (++t.tile < t.ntile) return;
  t.tile = 0;
  t.first = true;
  ++t.g;
  if (++t.kvh < p.n_kv_heads) return;
  t.kvh = 0;
  do {
    ++t.b;
    t.L = lens[t.b];
  } while (t.L <= 0);  // in range: tiles are left, so a later sequence has some
  t.ntile = dt_tiles(t.L);
}

// Reduction of eight values per lane over the 32 lanes of a warp with 9 shuffles instead of 40: at offsets 16, 8 and 4
// a lane hands half of its values to its partner and keeps the other half, then two plain butterfly steps.  Lane l ends
// up with the result for value index 4 (l >> 4 & 1) + 2 (l >> 3 & 1) + (l >> 2 & 1); lanes with l % 4 == 0 publish it.
template <bool MAX>
__device__ __forceinline__ float warp_reduce8(const float (&v)[8], int lane) {
  auto op = [](float a, float b) { return MAX ? fmaxf(a, b) : a + b; };
  const bool b4 = lane & 16, b3 = lane & 8, b2 = lane & 4;
  float a[4], c[2];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float send = b4 ? v[i] : v[4 + i], keep = b4 ? v[4 + i] : v[i];
    a[i] = op(keep, __shfl_xor_sync(0xffffffffu, send, 16));
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const float send = b3 ? a[i] : a[2 + i], keep = b3 ? a[2 + i] : a[i];
    c[i] = op(keep, __shfl_xor_sync(0xffffffffu, send, 8));
  }
  const float send = b2 ? c[0] : c[1], keep = b2 ? c[1] : c[0];
  float r = op(keep, __shfl_xor_sync(0xffffffffu, send, 4));
  r = op(r, __shfl_xor_sync(0xffffffffu, r, 2));
  r = op(r, __shfl_xor_sync(0xffffffffu, r, 1));
  return r;
}

__global__ void __launch_bounds__(kDThreads, 1)
decode_attention_tc_kernel(const DtParams p, const __grid_constant__ CUtensorMap map_k,
                           const __grid_constant__ CUtensorMap map_v) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t s_base = smem_u32(smem);
  float* red = reinterpret_cast<float*>(smem + OFF_STAT);  // [2 warpgroups][2 items][4 warps][8 heads] maxima per warp
  float* mst = red + 128;                                  // [4 items][8] maximum of the tile
  float* sst = mst + 32;                                   // [4 items][4 warps][8] sums per warp
  int* lens_s = reinterpret_cast<int*>(sst + 128);         // [batch] keys attended per sequence
  int* pre_s = lens_s + kMaxBatch;                         // [batch + 1] live tiles (x kv heads) of the sequences before
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_DBAR);
  uint64_t* k_full = bars;             // [3]
  uint64_t* k_empty = k_full + 3;      // [3]
  uint64_t* v_full = k_empty + 3;      // [3]
  uint64_t* v_empty = v_full + 3;      // [3]
  uint64_t* q_full = v_empty + 3;      // [2]
  uint64_t* q_empty = q_full + 2;      // [2]
  uint64_t* s_full = q_empty + 2;      // [2]
  uint64_t* s_empty = s_full + 2;      // [2]
  uint64_t* p_full = s_empty + 2;      // [2]: per softmax warpgroup (a warp cannot lap another: it waits for p_empty in between)
  uint64_t* p_empty = p_full + 2;      // [2]
  uint64_t* o_full = p_empty + 2;      // [2]
  uint64_t* o_empty = o_full + 2;      // [2]
  uint64_t* r_full = o_empty + 2;      // [2 warpgroups][2]: the warpgroup's four warps have written their maxima of an item
  uint64_t* st_full = r_full + 4;      // [4]: maximum and sums of an item are in shared memory (for the epilogue warps)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(st_full + 4);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int group = p.n_q_heads / p.n_kv_heads;  // query heads per kv head (<= 16)

  if (tid == 0) {
    for (int s = 0; s < 3; ++s) {
      mbar_init(&k_full[s], 1);
      mbar_init(&k_empty[s], 1);
      mbar_init(&v_full[s], 1);
      mbar_init(&v_empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&q_full[a], 1);
      mbar_init(&q_empty[a], 1);
      mbar_init(&s_full[a], 1);
      mbar_init(&s_empty[a], 4);
      mbar_init(&o_full[a], 1);
      mbar_init(&o_empty[a], 4);
      mbar_init(&p_full[a], 4);
      mbar_init(&p_empty[a], 1);
    }
    for (int a = 0; a < 4; ++a) {
      mbar_init(&st_full[a], 4);
      mbar_init(&r_full[a], 4);
    }
    fence_barrier_init();
  }
  if (warp == 13) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "n"(D_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // rows of P^T beyond the group's heads are never written: make them zero once (they feed unused output columns)
  for (int i = tid; i < 2 * Q_TILE / 16; i += kDThreads) sts128(s_base + OFF_P + i * 16, make_uint4(0, 0, 0, 0));
  fence_proxy_async();
  pdl_launch_dependents();
  pdl_wait();  // q, this step's key / value rows and the lengths come from the kernels before
  for (int b = tid; b < p.batch; b += kDThreads) lens_s[b] = max(0, min(p.kv_len[b] + p.kv_len_offset, p.max_seq_len));
  __syncthreads();
  if (warp == 0) {  // prefix of the live tiles: eight sequences per lane, then a scan over the lanes
    int own = 0;
    for (int j = 0; j < kMaxBatch / 32; ++j) {
      const int b = lane * (kMaxBatch / 32) + j;
      if (b < p.batch) own += dt_tiles(lens_s[b]) * p.n_kv_heads;
    }
    int incl = own;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += up;
    }
    int run = incl - own;
    for (int j = 0; j < kMaxBatch / 32; ++j) {
      const int b = lane * (kMaxBatch / 32) + j;
      if (b <= p.batch) pre_s[b] = run;
      if (b < p.batch) run += dt_tiles(lens_s[b]) * p.n_kv_heads;
    }
  }
  at_fence_before();
  __syncthreads();
  at_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_slot);

  if (warp == 12 || warp == 15) {
    // ------------------------------------------------------------------ TMA producers (warp 12: keys, warp 15: values)
    if (lane == 0) {
      const bool is_k = warp == 12;
      uint64_t* full = is_k ? k_full : v_full;
      uint64_t* empty = is_k ? k_empty : v_empty;
      const CUtensorMap* map = is_k ? &map_k : &map_v;
      const uint32_t ring = s_base + (is_k ? OFF_K : OFF_V);
      bool ok = true;
      DtItem t;
      dt_begin(p, lens_s, pre_s, t);
      int n = 0;
      for (; t.left > 0; ++n) {
        const int s = n % D_SLOTS;
        ok = at_wait(&empty[s], ((n / D_SLOTS) & 1) ^ 1u);
        if (!ok) break;
        const int row = (t.b * p.n_kv_heads + t.kvh) * p.max_seq_len + t.tile * kDT;
        mbar_expect_tx(&full[s], KV_TILE);
        for (int blk = 0; blk < 2; ++blk) at_tma_2d(ring + s * KV_TILE + blk * BLK_BYTES, map, blk * 64, row, &full[s]);
        dt_advance(p, lens_s, t);
      }
      if (!ok) {
        if (p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
        for (int j = 1; j <= D_SLOTS && j <= n; ++j)  // wait (bounded) for the copies still in flight
          at_wait(&full[(n - j) % D_SLOTS], ((n - j) / D_SLOTS) & 1);
      }
    }
  } else if (warp == 13) {
    // ------------------------------------------------------------------ MMA issuer of the scores
    if (lane == 0) {
      bool ok = true;
      DtItem t;
      dt_begin(p, lens_s, pre_s, t);
      for (int n = 0; t.left > 0; ++n) {  // S^T of the CTA's n-th live item
        const int s = n % D_SLOTS, sb = n & 1, qb = t.g & 1;
        ok = at_wait(&k_full[s], (n / D_SLOTS) & 1);
        if (ok && t.first) ok = at_wait(&q_full[qb], (t.g >> 1) & 1);  // the query tile of this (sequence, kv head)
        if (ok) ok = at_wait(&s_empty[sb], ((n >> 1) & 1) ^ 1u);
        if (!ok) break;
        at_fence_after();
        const uint64_t dk = desc_kmajor(s_base + OFF_K + s * KV_TILE);
        const uint64_t dq = desc_kmajor(s_base + OFF_Q + qb * Q_TILE);
        const uint32_t d_tmem = tmem_base + sb * 16;
#pragma unroll
        for (int k = 0; k < kDH / 16; ++k) {  // A: 64-column blocks of 16 KB; B: 64-column blocks of 2 KB (16 rows)
          const uint64_t offa = static_cast<uint64_t>((k >> 2) * (BLK_BYTES >> 4) + (k & 3) * 2);
          const uint64_t offb = static_cast<uint64_t>((k >> 2) * (2048 >> 4) + (k & 3) * 2);
          at_mma(d_tmem, dk + offa, dq + offb, IDESC_S, k > 0 ? 1u : 0u);
        }
        at_commit(&k_empty[s]);
        if (t.last_of_group()) at_commit(&q_empty[qb]);
        at_commit(&s_full[sb]);
        dt_advance(p, lens_s, t);
      }
      if (!ok && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
    }
  } else if (warp == 14) {
    // ------------------------------------------------------------------ MMA issuer of the P.V products
    if (lane == 0) {
      bool ok = true;
      DtItem t;
      dt_begin(p, lens_s, pre_s, t);
      for (int n = 0; t.left > 0; ++n) {  // O^T of the CTA's n-th live item
        const int s = n % D_SLOTS, ob = n & 1;
        ok = at_wait(&v_full[s], (n / D_SLOTS) & 1);
        if (ok) ok = at_wait(&p_full[ob], (n >> 1) & 1);
        if (ok) ok = at_wait(&o_empty[ob], ((n >> 1) & 1) ^ 1u);
        if (!ok) break;
        at_fence_after();
        const uint64_t dv = desc_mnmajor(s_base + OFF_V + s * KV_TILE);
        const uint64_t dp = desc_kmajor(s_base + OFF_P + ob * Q_TILE);  // the P^T of the warpgroup that had this item
        const uint32_t d_tmem = tmem_base + 32 + ob * 16;
#pragma unroll
        for (int k = 0; k < kDT / 16; ++k) {  // 16 keys per step: two 8-key atoms of V, 32 bytes along a row of P^T
          const uint64_t offb = static_cast<uint64_t>((k >> 2) * (2048 >> 4) + (k & 3) * 2);
          at_mma(d_tmem, dv + static_cast<uint64_t>(k * (2048 >> 4)), dp + offb, IDESC_O, k > 0 ? 1u : 0u);
        }
        at_commit(&v_empty[s]);
        at_commit(&p_empty[ob]);
        at_commit(&o_full[ob]);
        dt_advance(p, lens_s, t);
      }
      if (!ok && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
    }
  } else if (warp < 8) {
    // ------------------------------------------------------------------ softmax (warps 0..3 and 4..7; a thread = a key)
    const int wg = warp >> 2, wq = warp & 3;  // warpgroup (takes items n = wg, wg + 2, ...), TMEM lane quarter
    const int row = wq * 32 + lane;
    const float c = rsqrtf(static_cast<float>(kDH)) * 1.4426950408889634f;
    const int hsel = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);  // the head this lane reduces to
    bool ok = true;
    DtItem t;
    dt_begin(p, lens_s, pre_s, t);
    if (wg == 1 && t.left > 0) dt_advance(p, lens_s, t);
    for (int n = wg; t.left > 0; n += 2) {
      const int i = n >> 1;  // this warpgroup's i-th item
      const int slot = n % D_SLOTS;
      ok = at_wait_warp(&s_full[wg], i & 1);
      if (!ok) break;
      at_fence_after();
      uint32_t sr[16];
      at_ld16(tmem_base + (static_cast<uint32_t>(wq * 32) << 16) + wg * 16, sr);
      at_wait_ld();
      at_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_empty[wg]);
      const bool live = t.tile * kDT + row < t.L;  // this thread's key is attended
      float sv[8];
#pragma unroll
      for (int h = 0; h < 8; ++h)  // hi-part score + lo-part score
        sv[h] = live ? (__uint_as_float(sr[h]) + __uint_as_float(sr[8 + h])) * c : -INFINITY;
      // the four warps' maxima through shared memory: double-buffered by item, one bounded barrier per buffer (a warp
      // is at most one item ahead of another of its warpgroup: it needs every warp's arrival of the item before)
      float* rd = red + (wg * 2 + (i & 1)) * 32;
      uint64_t* rbar = &r_full[wg * 2 + (i & 1)];
      const float wm = warp_reduce8<true>(sv, lane);
      if ((lane & 3) == 0) rd[wq * 8 + hsel] = wm;
      __syncwarp();
      if (lane == 0) mbar_arrive(rbar);
      ok = at_wait_warp(rbar, (i >> 1) & 1);
      if (!ok) break;
      float e[8], mrow[8];
#pragma unroll
      for (int h = 0; h < 8; ++h) {
        mrow[h] = fmaxf(fmaxf(rd[h], rd[8 + h]), fmaxf(rd[16 + h], rd[24 + h]));  // finite: the tile's first key is live
        e[h] = ex2(sv[h] - mrow[h]);
      }
      const float su = warp_reduce8<false>(e, lane);
      // This warpgroup's previous P^T has been read.  The wait also guards the statistics ring below: the P.V product
      // of item n - 2 was issued only after the epilogue warps had released the output buffer of item n - 4, so slot
      // n % 4 of the ring (and its barrier) is no longer in use.  Without it the scores issuer, which no longer waits
      // for the P.V issuer, lets these warps run four items ahead of the epilogue.
      if (i > 0) ok = at_wait_warp(&p_empty[wg], (i - 1) & 1);
      if (!ok) break;
      float* ms = mst + (n & 3) * 8;
      float* ss = sst + ((n & 3) * 4 + wq) * 8;
      if (wq == 0 && lane < 8) {
        float mv = mrow[0];
#pragma unroll
        for (int h = 1; h < 8; ++h) mv = lane == h ? mrow[h] : mv;
        ms[lane] = mv;
      }
      if ((lane & 3) == 0) ss[hsel] = su;
      __syncwarp();
      if (lane == 0) mbar_arrive(&st_full[n & 3]);
      // P^T[head][key]: row = head for the hi part, 8 + head for the lo part (128 bytes per 64 keys, the 16-byte
      // chunks swizzled by row)
      {
        const int blk = row >> 6, col = row & 63;
        const uint32_t base = s_base + OFF_P + wg * Q_TILE + blk * 2048 + (col & 7) * 2;
#pragma unroll
        for (int h = 0; h < 8; ++h) {
          if (h >= group) break;
          const __half hi = __float2half_rn(e[h]);
          const __half lo = __float2half_rn(e[h] - __half2float(hi));
          const uint32_t a = base + h * 128 + (((col >> 3) ^ h) << 4);
          asm volatile("st.shared.u16 [%0], %1;" ::"r"(a), "h"(__half_as_ushort(hi)) : "memory");
          asm volatile("st.shared.u16 [%0], %1;" ::"r"(a + 8 * 128), "h"(__half_as_ushort(lo)) : "memory");
        }
      }
      if (t.tile * kDT + kDT > t.L) {  // the tile holds rows past the sequence's own: their value rows become zero
        ok = at_wait_warp(&v_full[slot], (n / D_SLOTS) & 1);  // once the tile has landed
        if (!ok) break;
      }
      if (!live) {
        const uint32_t vrow = s_base + OFF_V + slot * KV_TILE + row * 128;
#pragma unroll
        for (int blk = 0; blk < 2; ++blk)
#pragma unroll
          for (int ch = 0; ch < 8; ++ch) sts128(vrow + blk * BLK_BYTES + ch * 16, make_uint4(0, 0, 0, 0));
      }
      fence_proxy_async();  // the MMA reads P^T and V through the async proxy
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[wg]);
      dt_advance(p, lens_s, t);
      if (t.left > 0) dt_advance(p, lens_s, t);  // every other live item
    }
    if (!ok && lane == 0 && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
  } else if (warp == 16) {
    // ------------------------------------------------------------------ query conversion (one warp, a group ahead)
    // The query tile of a (sequence, kv head) group: its heads as rows 0-7 (binary16 hi part) and 8-15 (lo part) of
    // 128-byte swizzled blocks of 64 columns.  Two buffers: the scores issuer frees one with the group's last tile.
    bool ok = true;
    DtItem t;
    dt_begin(p, lens_s, pre_s, t);
    while (t.left > 0) {
      if (t.first) {
        const int qb = t.g & 1;
        ok = at_wait_warp(&q_empty[qb], ((t.g >> 1) & 1) ^ 1u);
        if (!ok) break;
        const float* src = p.q + (static_cast<size_t>(t.b) * p.n_q_heads + static_cast<size_t>(t.kvh) * group) * kDH;
        const uint32_t dst = s_base + OFF_Q + qb * Q_TILE;
#pragma unroll
        for (int j = 0; j < 4; ++j) {  // 8 rows x 16 chunks of 8 values, four chunks per lane
          const int i = j * 32 + lane, h = i >> 4, ch = i & 15;
          uint4 hi = make_uint4(0, 0, 0, 0), lo = hi;
          if (h < group) {
            const float4 a = __ldcg(reinterpret_cast<const float4*>(src + h * kDH + ch * 8));
            const float4 b2 = __ldcg(reinterpret_cast<const float4*>(src + h * kDH + ch * 8 + 4));
            const float v[8] = {a.x, a.y, a.z, a.w, b2.x, b2.y, b2.z, b2.w};
            uint32_t hw[4], lw[4];
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
              hw[jj] = pack_f16x2(v[2 * jj], v[2 * jj + 1]);
              lw[jj] = pack_f16x2(v[2 * jj] - f16_lo(hw[jj]), v[2 * jj + 1] - f16_hi(hw[jj]));
            }
            hi = make_uint4(hw[0], hw[1], hw[2], hw[3]);
            lo = make_uint4(lw[0], lw[1], lw[2], lw[3]);
          }
          const uint32_t a = dst + (ch >> 3) * 2048 + h * 128 + (((ch & 7) ^ h) << 4);  // lo: 8 rows further down
          sts128(a, hi);
          sts128(a + 8 * 128, lo);
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(&q_full[qb]);
      }
      dt_advance(p, lens_s, t);
    }
    if (!ok && lane == 0 && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
  } else {
    // ------------------------------------------------------------------ epilogue (warps 8..11)
    const int ew = warp - 8, d = ew * 32 + lane;  // this thread's output dimension = its TMEM lane
    constexpr int stride = kDH + 2;
    bool ok = true;
    // empty partials for the tiles beyond a sequence's length (dealt round-robin over the CTAs)
    for (int w = blockIdx.x; w < p.n_items; w += gridDim.x) {
      const int tile = w % p.n_tiles, r = w / p.n_tiles, kvh = r % p.n_kv_heads, b = r / p.n_kv_heads;
      if (tile * kDT < lens_s[b]) continue;
      for (int h = 0; h < group; ++h) {
        float* dst = p.scratch + ((static_cast<size_t>(b) * p.n_q_heads + kvh * group + h) * p.n_tiles + tile) * stride;
        dst[d] = 0.f;
        if (d == 0) {
          dst[kDH] = -INFINITY;
          dst[kDH + 1] = 0.f;
        }
      }
    }
    DtItem t;
    dt_begin(p, lens_s, pre_s, t);
    for (int n = 0; t.left > 0; ++n) {
      const int ob = n & 1;
      ok = at_wait_warp(&st_full[n & 3], (n >> 2) & 1);
      if (ok) ok = at_wait_warp(&o_full[ob], (n >> 1) & 1);
      if (!ok) break;
      at_fence_after();
      uint32_t orr[16];
      at_ld16(tmem_base + (static_cast<uint32_t>(ew * 32) << 16) + 32 + ob * 16, orr);
      at_wait_ld();
      const float* ms = mst + (n & 3) * 8;
      const float* ss = sst + (n & 3) * 32;
      float mh = 0.f, lh = 0.f;
      if (d < group) {
        mh = ms[d] * 0.6931471805599453f;  // the softmax warps work in base 2; the merge kernel expects natural logarithms
        lh = (ss[d] + ss[8 + d]) + (ss[16 + d] + ss[24 + d]);
      }
      at_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&o_empty[ob]);  // O^T and the statistics of this item have been read
#pragma unroll
      for (int h = 0; h < kNH; ++h) {
        if (h >= group) break;
        float* dst = p.scratch + ((static_cast<size_t>(t.b) * p.n_q_heads + t.kvh * group + h) * p.n_tiles + t.tile) * stride;
        dst[d] = __uint_as_float(orr[h]) + __uint_as_float(orr[8 + h]);  // P hi part + P lo part
      }
      if (d < group) {
        float* dst = p.scratch + ((static_cast<size_t>(t.b) * p.n_q_heads + t.kvh * group + d) * p.n_tiles + t.tile) * stride;
        dst[kDH] = mh;
        dst[kDH + 1] = lh;
      }
      dt_advance(p, lens_s, t);
    }
    if (!ok && lane == 0 && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
  }

  at_fence_before();
  __syncthreads();
  if (warp == 13) {
    at_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(D_TMEM_COLS) : "memory");
  }
}

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn g_dt_encode = nullptr;
int g_dt_sms = 0;

cudaError_t dt_make_map(CUtensorMap* map, const void* base, uint64_t rows) {
  const cuuint64_t dims[2] = {kDH, rows};
  const cuuint64_t strides[1] = {kDH * 2};
  const cuuint32_t box[2] = {64, 128};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = g_dt_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

}  // namespace

cudaError_t decode_attention_tc_init() {
  if (!g_dt_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    g_dt_encode = reinterpret_cast<EncodeFn>(fn);
  }
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&g_dt_sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(decode_attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, D_SMEM);
}

bool decode_attention_tc_usable(const DecodeAttnParams& p) {  // the shapes the kernel handles
  return p.head_dim == kDH && p.n_q_heads / p.n_kv_heads <= kNH && p.batch <= kMaxBatch;
}

// The split kernel of the wide-batch path: one partial per 128 keys into p.scratch, laid out [batch][Hq][n_tiles][130].
cudaError_t launch_decode_attention_tc(const DecodeAttnParams& p, int n_tiles, int32_t* status, cudaStream_t stream,
                                       bool pdl) {
  if (!decode_attention_tc_usable(p) || n_tiles < 1) return cudaErrorInvalidValue;
  if (!g_dt_encode) {  // an op-level caller that did not go through model creation: set up on first use (no allocation)
    const cudaError_t ei = decode_attention_tc_init();
    if (ei != cudaSuccess) return ei;
  }
  CUtensorMap mk, mv;
  const uint64_t rows = static_cast<uint64_t>(p.batch) * p.n_kv_heads * p.max_seq_len;
  cudaError_t e = dt_make_map(&mk, p.k, rows);
  if (e == cudaSuccess) e = dt_make_map(&mv, p.v, rows);
  if (e != cudaSuccess) return e;
  DtParams d = {};
  d.q = p.q;
  d.kv_len = p.kv_len;
  d.kv_len_offset = p.kv_len_offset;
  d.batch = p.batch;
  d.n_q_heads = p.n_q_heads;
  d.n_kv_heads = p.n_kv_heads;
  d.max_seq_len = p.max_seq_len;
  d.n_tiles = n_tiles;
  d.n_items = p.batch * p.n_kv_heads * n_tiles;
  d.scratch = p.scratch;
  d.status = status;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(d.n_items < g_dt_sms ? d.n_items : g_dt_sms);
  cfg.blockDim = dim3(kDThreads);
  cfg.dynamicSmemBytes = D_SMEM;
  cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, decode_attention_tc_kernel, d, mk, mv);
}

}  // namespace ladder
