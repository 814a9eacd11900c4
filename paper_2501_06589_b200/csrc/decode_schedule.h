// Batch schedule of the weight-streaming decode GEMM (host side, shared by the per-GEMM kernel and
// the persistent layer-stack kernel).  The rows of W are cut into 8-row units; claim i of a GEMM
// maps to a run of consecutive units by this fixed table, so claiming is a single atomicAdd.
#pragma once

namespace ladder {

constexpr int kSchedMaxPhases = 24;
constexpr int kSchedUnitsMax = 10;  // 8-row units per claim at most (5 MMA row groups)

// Round i hands out count[i] claims of size[i] consecutive units.
struct Schedule {
  int n;
  int count[kSchedMaxPhases];
  int size[kSchedMaxPhases];
  // The first n_static claims can be dealt out without the counter, claim i to CTA i % grid (whole
  // rounds of one claim per CTA); only the claims after them need to be taken dynamically.
  int n_static;
  int n_claims;  // all claims
};

// A batch costs a fixed latency per K chunk (activation hand-over, fragment hoisting) and re-reads
// the activations, so small batches are expensive; but equal static shares make every launch wait
// for the slowest SM.  Hence:
//   * little work per CTA (share <= kSchedUnitsMax units): one round of near-equal batches, each done
//     in a single pass over K (measured faster than a 70 % + 30 % split, whose second pass is too short);
//   * more: rounds of 8-unit batches while a CTA's share of what is left is large, then one round
//     of ~70 % of the remaining share, then 2-unit batches with which the fast SMs pick up the
//     slack of the slow ones (guided self-scheduling, evaluated ahead of time).
inline Schedule make_schedule(int n_units, int grid) {
  Schedule sc = {};
  auto push = [&](int count, int size) {
    if (count <= 0 || size <= 0) return;
    if (sc.n > 0 && sc.size[sc.n - 1] == size) {  // same size as the round before: one longer round
      sc.count[sc.n - 1] += count;
    } else if (sc.n < kSchedMaxPhases) {
      sc.count[sc.n] = count;
      sc.size[sc.n] = size;
      ++sc.n;
    }
  };
  int rem = n_units;
  if (rem <= kSchedUnitsMax * grid) {
    const int hi = (rem + grid - 1) / grid, n_hi = rem - (hi - 1) * grid;  // n_hi batches of hi, rest hi-1
    push(n_hi, hi);
    push(grid - n_hi, hi - 1);
    sc.n_claims = hi > 1 ? grid : n_hi;
    sc.n_static = sc.n_claims;
    return sc;
  }
  while (rem > 0 && sc.n < kSchedMaxPhases - 2) {
    const double share = static_cast<double>(rem) / grid;
    int size;
    constexpr int kBig = kSchedUnitsMax < 8 ? kSchedUnitsMax : 8;
    if (share >= 12.0) size = kBig;
    else if (share >= 4.0) size = (static_cast<int>(share * 0.7) & ~1) > kBig ? kBig : (static_cast<int>(share * 0.7) & ~1);
    else break;
    push(grid, size);
    rem -= grid * size;
    sc.n_static += grid;
  }
  push(rem / 2, 2);
  push(rem & 1, 1);
  sc.n_claims = sc.n_static + rem / 2 + (rem & 1);
  return sc;
}

}  // namespace ladder
