// Causal grouped-query attention of the prompt pass on the 5th-generation tensor cores (tcgen05, sm_100a).
//
// Work item = (128-query tile, query head, sequence).  Persistent CTAs, one per SM; CTA c takes items c, c + grid,
// c + 2 grid, ... of a list ordered longest first, and treats the key tiles of all its items as ONE sequence of
// tiles, so the pipeline below never drains between items (a CTA per item spent more time filling and draining the
// pipeline than computing at 1024-token prompts).  320 threads in four roles that meet only at mbarriers:
//   warp 0      TMA producer: the query tile of an item (double-buffered when the query has no lo part), and
//               key / value tiles of 128 cache rows in the order the tensor core consumes them (K0, K1, V0, K2,
//               V1, ...) into a ring of four shared-memory slots (cp.async.bulk.tensor.2d, 128-byte swizzle; rows
//               beyond the tensor are zero-filled);
//   warp 1      MMA issuer: one thread issues tcgen05.mma (kind::f16, binary16 operands, fp32 accumulators in
//               tensor memory).  S = Q K^T (M 128, N 128, K = head_dim; the query's lo part adds a second round)
//               goes into one of two S buffers, so the scores of the next tile are computed while the softmax warps
//               work on this one; then PV = P V (M 128, N = head_dim, K 128) with P read from tensor memory and V
//               straight from the cache layout as an MN-major shared-memory operand, into one of two PV buffers;
//   warps 2-5   softmax: a thread owns one query row; it reads the row of S with tcgen05.ld, applies scale and the
//               causal mask, keeps the running maximum and sum, and writes P as binary16 over the first half of
//               the S buffer (tcgen05.st) together with the row's rescaling factor (shared memory);
//   warps 6-9   accumulate: a thread owns the same query row of the output; per tile it reads PV from tensor
//               memory and forms O = O * factor + PV in registers; after an item's last tile it divides by the row
//               sum and stores the row (binary16, or a bf16 hi + lo pair).
// Query p attends cache rows t <= p; query head h uses kv head h / (Hq / Hkv).  Value rows of an item's last tile
// that lie beyond the rows the sequence owns are zeroed in shared memory before the MMA reads them (their
// probabilities are zero, but stale cache bytes could hold NaN).  Every wait is bounded; on a protocol error the
// kernel records it in the status word, drains its copies and frees its tensor memory.
#include <cuda.h>

#include "common.cuh"
#include "kernels.h"
#include "tcgen05_attn.cuh"

namespace ladder {
namespace {

constexpr int kQT = 128, kKT = 128, kAtThreads = 320;

template <int DH, bool SPLIT>
struct AtCfg {
  static constexpr int NBLK = DH / 64;                  // 64-column blocks per query / key / value row
  static constexpr int TILE_BYTES = NBLK * BLK_BYTES;   // a Q, K or V tile
  static constexpr int SLOTS = 4;
  static constexpr int QBUF = SPLIT ? 1 : 2;            // query buffers (each: hi, and lo when SPLIT)
  static constexpr int Q_BYTES = (SPLIT ? 2 : 1) * TILE_BYTES;
  static constexpr int OFF_RING = QBUF * Q_BYTES;
  static constexpr int OFF_FACT = OFF_RING + SLOTS * TILE_BYTES;  // float factor[4][128], float rowsum[4][128]
  static constexpr int OFF_BARS = OFF_FACT + 8 * 128 * 4;
  static constexpr int SMEM = OFF_BARS + 32 * 8 + 1024;
  // Instruction descriptors, kind::f16 with binary16 A and B (format 0), fp32 D (bit 4), N >> 3 at bit 17,
  // M >> 4 at bit 24; bit 16 set = B is MN-major (the value tile: head_dim contiguous, keys strided).
  static constexpr uint32_t IDESC_QK = (1u << 4) | (static_cast<uint32_t>(kKT >> 3) << 17) |
                                       (static_cast<uint32_t>(kQT >> 4) << 24);
  static constexpr uint32_t IDESC_PV = (1u << 4) | (1u << 16) | (static_cast<uint32_t>(DH >> 3) << 17) |
                                       (static_cast<uint32_t>(kQT >> 4) << 24);
  static constexpr int TMEM_COLS = 512;  // S0, S1 at 0 / 128 (P_j overwrites the first 64 columns of S_j); PV0, PV1 at 256 / 384
};

struct AtParams {
  int seq_len, n_q_heads, n_kv_heads, max_seq_len, pos0, out_f16, n_qt, batch, n_items;
  const int32_t* lens;
  __nv_bfloat16* o;
  __nv_bfloat16* o_lo;
  int32_t* status;
};

// One (work item, key tile) of a CTA's tile sequence.  Every role walks the same sequence with its own copy.
struct AtTile {
  int w;            // work item; >= n_items: the sequence is over
  int j, n_kt;      // key tile, and the item's number of key tiles
  int h, b, q0, len_b;
};
__device__ __forceinline__ bool at_item(const AtParams& p, int w, AtTile& t) {
  // items ordered longest first (late query tiles), heads of one kv group side by side
  const int per = p.n_q_heads * p.batch;
  const int qt = p.n_qt - 1 - w / per, rest = w % per;
  t.b = rest / p.n_q_heads;
  t.h = rest % p.n_q_heads;
  t.q0 = qt * kQT;
  t.len_b = p.lens ? min(max(p.lens[t.b], 0), p.seq_len) : p.seq_len;
  if (t.q0 >= t.len_b) return false;  // a tile of padding rows
  const int q_hi = min(t.q0 + kQT, t.len_b) - 1;  // last valid query of the tile
  t.n_kt = (p.pos0 + q_hi) / kKT + 1;             // key tiles this query tile attends to
  t.j = 0;
  t.w = w;
  return true;
}
__device__ __forceinline__ void at_seek(const AtParams& p, int w, AtTile& t) {
  while (w < p.n_items && !at_item(p, w, t)) w += gridDim.x;
  if (w >= p.n_items) t.w = p.n_items;
}
__device__ __forceinline__ void at_first(const AtParams& p, AtTile& t) { at_seek(p, blockIdx.x, t); }
__device__ __forceinline__ void at_next(const AtParams& p, AtTile& t) {
  if (++t.j < t.n_kt) return;
  at_seek(p, t.w + gridDim.x, t);
}

template <int DH, bool SPLIT>
__global__ void __launch_bounds__(kAtThreads, 1)
prefill_attention_tc_kernel(const AtParams p, const __grid_constant__ CUtensorMap map_q,
                            const __grid_constant__ CUtensorMap map_qlo, const __grid_constant__ CUtensorMap map_k,
                            const __grid_constant__ CUtensorMap map_v) {
  using C = AtCfg<DH, SPLIT>;
  constexpr int SLOTS = C::SLOTS, NBLK = C::NBLK, TILE_BYTES = C::TILE_BYTES, QBUF = C::QBUF;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t s_base = smem_u32(smem);
  float* fact = reinterpret_cast<float*>(smem + C::OFF_FACT);  // [4][128] rescaling factor of a tile
  float* lsum = fact + 4 * 128;                                // [4][128] row sums, written with an item's last tile
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BARS);
  uint64_t* q_full = bars;              // [2]
  uint64_t* q_empty = q_full + 2;       // [2]
  uint64_t* kv_full = q_empty + 2;      // [SLOTS]
  uint64_t* kv_empty = kv_full + SLOTS;
  uint64_t* s_full = kv_empty + SLOTS;  // [2]
  uint64_t* s_empty = s_full + 2;
  uint64_t* p_full = s_empty + 2;       // [2]: one per S buffer.  With a single barrier a softmax warp one tile ahead
                                        // of another (the next scores are ready early) would arrive twice in one phase
  uint64_t* pv_full = p_full + 2;       // [2]
  uint64_t* pv_empty = pv_full + 2;
  uint64_t* f_full = pv_empty + 2;      // [4]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(f_full + 4);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int group = p.n_q_heads / p.n_kv_heads;

  if (tid == 0) {
    for (int a = 0; a < 2; ++a) {
      mbar_init(&q_full[a], 1);
      mbar_init(&q_empty[a], 1);
      mbar_init(&s_full[a], 1);
      mbar_init(&s_empty[a], 4);
      mbar_init(&pv_full[a], 1);
      mbar_init(&pv_empty[a], 4);
      mbar_init(&p_full[a], 4);
    }
    for (int s = 0; s < SLOTS; ++s) {
      mbar_init(&kv_full[s], 1);
      mbar_init(&kv_empty[s], 1);
    }
    for (int a = 0; a < 4; ++a) mbar_init(&f_full[a], 4);
    fence_barrier_init();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "n"(C::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  at_fence_before();
  __syncthreads();
  at_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_slot);

  // Ring position of the tiles of the sequence: K of tile 0 is copy 0; K of tile g > 0 is copy 2g - 1; V of tile g
  // is copy 2g + 2 when a tile g + 1 follows (its K is fetched first), else copy 2g + 1.
  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      bool ok = true;
      int it = 0, n = 0;
      auto load_q = [&](const AtTile& t) {  // the query tile of item number n
        const int qb = n % QBUF;
        ok = at_wait(&q_empty[qb], ((n / QBUF) & 1) ^ 1u);
        if (!ok) return;
        mbar_expect_tx(&q_full[qb], C::Q_BYTES);
        const uint32_t dst = s_base + qb * C::Q_BYTES;
        for (int blk = 0; blk < NBLK; ++blk) {
          at_tma_2d(dst + blk * BLK_BYTES, &map_q, t.h * DH + blk * 64, t.b * p.seq_len + t.q0, &q_full[qb]);
          if (SPLIT)
            at_tma_2d(dst + TILE_BYTES + blk * BLK_BYTES, &map_qlo, t.h * DH + blk * 64, t.b * p.seq_len + t.q0,
                      &q_full[qb]);
        }
      };
      auto load_kv = [&](const CUtensorMap* map, const AtTile& t) {
        if (!ok) return;
        const int s = it % SLOTS;
        ok = at_wait(&kv_empty[s], ((it / SLOTS) & 1) ^ 1u);
        if (!ok) return;
        const int row = (t.b * p.n_kv_heads + t.h / group) * p.max_seq_len + t.j * kKT;
        mbar_expect_tx(&kv_full[s], TILE_BYTES);
        for (int blk = 0; blk < NBLK; ++blk)
          at_tma_2d(s_base + C::OFF_RING + s * TILE_BYTES + blk * BLK_BYTES, map, blk * 64, row, &kv_full[s]);
        ++it;
      };
      AtTile cur;
      at_first(p, cur);
      if (cur.w < p.n_items) {
        load_q(cur);
        load_kv(&map_k, cur);
      }
      while (cur.w < p.n_items && ok) {
        AtTile nxt = cur;
        at_next(p, nxt);
        if (nxt.w < p.n_items) {
          if (nxt.j == 0) {
            ++n;
            load_q(nxt);
          }
          load_kv(&map_k, nxt);
        }
        load_kv(&map_v, cur);
        cur = nxt;
      }
      if (!ok) {
        if (p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
        for (int j = 1; j <= SLOTS && j <= it; ++j) {  // wait (bounded) for the copies still in flight
          const int i2 = it - j;
          at_wait(&kv_full[i2 % SLOTS], (i2 / SLOTS) & 1);
        }
        for (int j = 0; j < QBUF && j <= n; ++j) at_wait(&q_full[(n - j) % QBUF], ((n - j) / QBUF) & 1);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = true;
      int it = 0, n = 0;
      auto scores = [&](const AtTile& t, int g) {  // S = Q K^T of tile g (item number n) into S buffer g & 1
        const int s = it % SLOTS, sb = g & 1, qb = n % QBUF;
        if (t.j == 0) ok = at_wait(&q_full[qb], (n / QBUF) & 1);
        if (ok) ok = at_wait(&kv_full[s], (it / SLOTS) & 1);
        if (ok) ok = at_wait(&s_empty[sb], ((g >> 1) & 1) ^ 1u);
        if (!ok) return;
        at_fence_after();
        const uint64_t dq = desc_kmajor(s_base + qb * C::Q_BYTES), dql = desc_kmajor(s_base + qb * C::Q_BYTES + TILE_BYTES);
        const uint64_t dk = desc_kmajor(s_base + C::OFF_RING + s * TILE_BYTES);
        const uint32_t d_tmem = tmem_base + sb * 128;
#pragma unroll
        for (int k = 0; k < DH / 16; ++k) {  // +32 bytes along the swizzled row = +2 in the address field
          const uint64_t off = static_cast<uint64_t>((k >> 2) * (BLK_BYTES >> 4) + (k & 3) * 2);
          at_mma(d_tmem, dq + off, dk + off, C::IDESC_QK, k > 0 ? 1u : 0u);
        }
        if (SPLIT) {
#pragma unroll
          for (int k = 0; k < DH / 16; ++k) {
            const uint64_t off = static_cast<uint64_t>((k >> 2) * (BLK_BYTES >> 4) + (k & 3) * 2);
            at_mma(d_tmem, dql + off, dk + off, C::IDESC_QK, 1u);
          }
        }
        at_commit(&kv_empty[s]);
        if (t.j == t.n_kt - 1) at_commit(&q_empty[qb]);  // the item's last use of its query tile
        at_commit(&s_full[sb]);
        ++it;
      };
      AtTile cur;
      at_first(p, cur);
      int g = 0;
      if (cur.w < p.n_items) scores(cur, 0);
      while (cur.w < p.n_items && ok) {
        AtTile nxt = cur;
        at_next(p, nxt);
        if (nxt.w < p.n_items) {
          if (nxt.j == 0) ++n;
          scores(nxt, g + 1);
          if (!ok) break;
        }
        const int s = it % SLOTS, ob = g & 1;  // PV = P V of tile g into PV buffer g & 1
        ok = at_wait(&kv_full[s], (it / SLOTS) & 1);
        if (ok) ok = at_wait(&p_full[ob], (g >> 1) & 1);
        if (ok) ok = at_wait(&pv_empty[ob], ((g >> 1) & 1) ^ 1u);
        if (!ok) break;
        at_fence_after();
        const uint64_t dv = desc_mnmajor(s_base + C::OFF_RING + s * TILE_BYTES);
        const uint32_t d_tmem = tmem_base + 256 + ob * 128;
#pragma unroll
        for (int k = 0; k < kKT / 16; ++k)  // 16 keys per step: 8 packed columns of P, two 8-key atoms of V
          at_mma_ts(d_tmem, tmem_base + ob * 128 + k * 8, dv + static_cast<uint64_t>(k * (2048 >> 4)), C::IDESC_PV,
                    k > 0 ? 1u : 0u);
        at_commit(&kv_empty[s]);
        at_commit(&pv_full[ob]);
        ++it;
        cur = nxt;
        ++g;
      }
      if (!ok && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------------ softmax (warps 2..5)
    const int qd = warp & 3, row = qd * 32 + lane;  // the TMEM lane quarter this warp may access
    const float c = rsqrtf(static_cast<float>(DH)) * 1.4426950408889634f;
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = true;
    AtTile cur;
    at_first(p, cur);
    for (int g = 0; cur.w < p.n_items; ++g) {
      if (cur.j == 0) {
        m_run = -INFINITY;
        l_run = 0.f;
      }
      const int sb = g & 1, k0 = cur.j * kKT;
      const int qpos = p.pos0 + cur.q0 + row;
      ok = at_wait_warp(&s_full[sb], (g >> 1) & 1);
      if (!ok) break;
      at_fence_after();
      uint32_t s[128];
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(qd * 32) << 16) + sb * 128;
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) at_ld32(taddr + cc * 32, s + cc * 32);
      at_wait_ld();
      at_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_empty[sb]);

      // four independent chains for the maximum and the sum: one warp per scheduler has no other warp to hide
      // the latency of a dependent chain behind
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      if (k0 + kKT - 1 > p.pos0 + cur.q0) {  // the tile reaches past the tile's first query: mask keys after the row's own
#pragma unroll
        for (int i = 0; i < 128; ++i) {
          const float v = (k0 + i <= qpos) ? __uint_as_float(s[i]) : -INFINITY;
          s[i] = __float_as_uint(v);
          mx4[i & 3] = fmaxf(mx4[i & 3], v);
        }
      } else {
#pragma unroll
        for (int i = 0; i < 128; ++i) mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(s[i]));
      }
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      const float m_new = fmaxf(m_run, mx * c);
      const float m_ref = (m_new == -INFINITY) ? 0.f : m_new;
      const float corr = ex2(m_run - m_ref);  // 0 for an item's first tile
      m_run = m_new;
      float sum4[4] = {0.f, 0.f, 0.f, 0.f};
      uint32_t pk[64];
#pragma unroll
      for (int i = 0; i < 64; ++i) {
        const float e0 = ex2(fmaf(__uint_as_float(s[2 * i]), c, -m_ref));
        const float e1 = ex2(fmaf(__uint_as_float(s[2 * i + 1]), c, -m_ref));
        sum4[i & 3] += e0 + e1;
        pk[i] = pack_f16x2(e0, e1);
      }
      const float sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
      l_run = l_run * corr + sum;

      // P over the first 64 columns of this S buffer (read into registers above; the buffer is written again by the
      // scores of tile g+2, which the tensor core starts after the P.V MMAs of tile g)
      at_st32(taddr, pk);
      at_st32(taddr + 32, pk + 32);
      fact[(g & 3) * 128 + row] = corr;
      if (cur.j == cur.n_kt - 1) {
        lsum[(g & 3) * 128 + row] = l_run;
        const int n_keys = p.pos0 + cur.len_b;  // cache rows this sequence owns after the call
        if (k0 + kKT > n_keys) {               // value rows past the sequence's own: make them zero
          AtTile nxt = cur;
          at_next(p, nxt);
          const int itv = nxt.w < p.n_items ? 2 * g + 2 : 2 * g + 1, sv = itv % SLOTS;
          ok = at_wait_warp(&kv_full[sv], (itv / SLOTS) & 1);
          if (!ok) break;
          if (k0 + row >= n_keys) {
            const uint32_t vrow = s_base + C::OFF_RING + sv * TILE_BYTES + row * 128;
#pragma unroll
            for (int blk = 0; blk < NBLK; ++blk)
#pragma unroll
              for (int ch = 0; ch < 8; ++ch) sts128(vrow + blk * BLK_BYTES + ch * 16, make_uint4(0, 0, 0, 0));
          }
          fence_proxy_async();  // the MMA reads V through the async proxy
        }
      }
      at_wait_st();
      at_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&p_full[sb]);
        mbar_arrive(&f_full[g & 3]);
      }
      at_next(p, cur);
    }
    if (!ok && lane == 0 && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
  } else {
    // ------------------------------------------------------------------ accumulate (warps 6..9)
    const int qd = warp & 3, row = qd * 32 + lane;
    float o[DH];
    bool ok = true;
    AtTile cur;
    at_first(p, cur);
    for (int g = 0; cur.w < p.n_items; ++g) {
      if (cur.j == 0) {
#pragma unroll
        for (int i = 0; i < DH; ++i) o[i] = 0.f;
      }
      const int ob = g & 1;
      ok = at_wait_warp(&f_full[g & 3], (g >> 2) & 1);
      if (ok) ok = at_wait_warp(&pv_full[ob], (g >> 1) & 1);
      if (!ok) break;
      at_fence_after();
      const float corr = fact[(g & 3) * 128 + row];
      const bool last = cur.j == cur.n_kt - 1;
      const float l = last ? lsum[(g & 3) * 128 + row] : 1.f;
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(qd * 32) << 16) + 256 + ob * 128;
#pragma unroll
      for (int cc = 0; cc < DH / 32; ++cc) {
        uint32_t r[32];
        at_ld32(taddr + cc * 32, r);
        at_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) o[cc * 32 + i] = fmaf(o[cc * 32 + i], corr, __uint_as_float(r[i]));
      }
      at_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&pv_empty[ob]);  // factor, row sum and PV of this tile have been read
      if (last) {
        const float inv = l > 0.f ? 1.f / l : 0.f;
        const int qi = cur.q0 + row;
        if (qi < cur.len_b) {
          const size_t doff = (static_cast<size_t>(cur.b) * p.seq_len + qi) * (static_cast<size_t>(p.n_q_heads) * DH) +
                              static_cast<size_t>(cur.h) * DH;
          if (p.out_f16) {  // one binary16 value per element: the operand of the binary16 output projection
            uint4* dst = reinterpret_cast<uint4*>(p.o + doff);
#pragma unroll
            for (int i = 0; i < DH / 8; ++i)
              dst[i] = make_uint4(pack_f16x2(o[8 * i] * inv, o[8 * i + 1] * inv), pack_f16x2(o[8 * i + 2] * inv, o[8 * i + 3] * inv),
                                  pack_f16x2(o[8 * i + 4] * inv, o[8 * i + 5] * inv), pack_f16x2(o[8 * i + 6] * inv, o[8 * i + 7] * inv));
          } else {
            uint4* dst = reinterpret_cast<uint4*>(p.o + doff);
            uint4* dst_lo = p.o_lo ? reinterpret_cast<uint4*>(p.o_lo + doff) : nullptr;
#pragma unroll
            for (int i = 0; i < DH / 8; ++i) {
              uint32_t hi[4], lo[4];
#pragma unroll
              for (int w = 0; w < 4; ++w) {
                const float v0 = o[8 * i + 2 * w] * inv, v1 = o[8 * i + 2 * w + 1] * inv;
                hi[w] = pack_bf16x2(v0, v1);
                lo[w] = pack_bf16x2(v0 - bf16_lo(hi[w]), v1 - bf16_hi(hi[w]));
              }
              dst[i] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
              if (dst_lo) dst_lo[i] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            }
          }
        }
      }
      at_next(p, cur);
    }
    if (!ok && lane == 0 && p.status) atomicOr(p.status, LADDER_DEV_TIMEOUT);
  }

  at_fence_before();
  __syncthreads();
  if (warp == 1) {
    at_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(C::TMEM_COLS) : "memory");
  }
}

// ---------------------------------------------------------------- host: tensor maps
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn g_at_encode = nullptr;
int g_at_sms = 0;  // CTAs of a launch: one per SM

// rows x cols binary16, row-major with `pitch` elements between rows; boxes of 128 rows x 64 columns
cudaError_t at_make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {pitch * 2};
  const cuuint32_t box[2] = {64, 128};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = g_at_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                                 estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int DH, bool SPLIT>
cudaError_t at_launch(const AtParams& p, const __half* q, const __half* q_lo, const kv_t* k, const kv_t* v, int batch,
                      cudaStream_t stream) {
  CUtensorMap mq, ml, mk, mv;
  const uint64_t qcols = static_cast<uint64_t>(p.n_q_heads) * DH, qrows = static_cast<uint64_t>(batch) * p.seq_len;
  const uint64_t kvrows = static_cast<uint64_t>(batch) * p.n_kv_heads * p.max_seq_len;
  cudaError_t e = at_make_map(&mq, q, qrows, qcols, qcols);
  if (e == cudaSuccess) e = at_make_map(&ml, SPLIT ? q_lo : q, qrows, qcols, qcols);
  if (e == cudaSuccess) e = at_make_map(&mk, k, kvrows, DH, DH);
  if (e == cudaSuccess) e = at_make_map(&mv, v, kvrows, DH, DH);
  if (e != cudaSuccess) return e;
  const int grid = p.n_items < g_at_sms ? p.n_items : g_at_sms;
  prefill_attention_tc_kernel<DH, SPLIT><<<grid, kAtThreads, AtCfg<DH, SPLIT>::SMEM, stream>>>(p, mq, ml, mk, mv);
  return cudaGetLastError();
}

template <int DH, bool SPLIT>
cudaError_t at_init() {
  return cudaFuncSetAttribute(prefill_attention_tc_kernel<DH, SPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              AtCfg<DH, SPLIT>::SMEM);
}

}  // namespace

cudaError_t prefill_attention_tc_init() {
  if (!g_at_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    g_at_encode = reinterpret_cast<EncodeFn>(fn);
  }
  int dev = 0;
  cudaError_t ed = cudaGetDevice(&dev);
  if (ed == cudaSuccess) ed = cudaDeviceGetAttribute(&g_at_sms, cudaDevAttrMultiProcessorCount, dev);
  if (ed != cudaSuccess) return ed;
  if (g_at_sms < 1) return cudaErrorNotSupported;
  cudaError_t e = at_init<128, true>();
  if (e == cudaSuccess) e = at_init<128, false>();
  if (e == cudaSuccess) e = at_init<64, true>();
  if (e == cudaSuccess) e = at_init<64, false>();
  return e;
}

cudaError_t launch_prefill_attention(const __half* q, const __half* q_lo, const kv_t* k, const kv_t* v, int batch,
                                     int seq_len, int n_q_heads, int n_kv_heads, int head_dim, int max_seq_len,
                                     __nv_bfloat16* o, __nv_bfloat16* o_lo, cudaStream_t stream, int pos0,
                                     bool out_f16, const int32_t* lens, int32_t* status) {
  if (!g_at_encode) return cudaErrorNotReady;
  if (out_f16 && o_lo) return cudaErrorInvalidValue;
  if (pos0 < 0 || pos0 + seq_len > max_seq_len) return cudaErrorInvalidValue;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(q_lo) | reinterpret_cast<uintptr_t>(k) |
       reinterpret_cast<uintptr_t>(v) | reinterpret_cast<uintptr_t>(o) | reinterpret_cast<uintptr_t>(o_lo)) & 15)
    return cudaErrorMisalignedAddress;
  const bool split = q_lo != nullptr && (o_lo != nullptr || out_f16);
  AtParams p = {};
  p.seq_len = seq_len;
  p.n_q_heads = n_q_heads;
  p.n_kv_heads = n_kv_heads;
  p.max_seq_len = max_seq_len;
  p.pos0 = pos0;
  p.out_f16 = out_f16 ? 1 : 0;
  p.n_qt = (seq_len + kQT - 1) / kQT;
  p.batch = batch;
  p.n_items = p.n_qt * n_q_heads * batch;
  p.lens = lens;
  p.o = o;
  p.o_lo = split ? o_lo : nullptr;
  p.status = status;
  if (head_dim == 128)
    return split ? at_launch<128, true>(p, q, q_lo, k, v, batch, stream) : at_launch<128, false>(p, q, q_lo, k, v, batch, stream);
  if (head_dim == 64)
    return split ? at_launch<64, true>(p, q, q_lo, k, v, batch, stream) : at_launch<64, false>(p, q, q_lo, k, v, batch, stream);
  return cudaErrorInvalidValue;
}

}  // namespace ladder
