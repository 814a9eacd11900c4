// Tensor-parallel exchange over peer memory (paper Sec. 2, Eq. 1: the all-reduce of a module's partial sums;
// Algorithm 1 overlaps it with the next module).  For the decode step's messages ([batch, d_model] fp32: 32 KiB to
// 2 MiB) a ring or tree pays several link latencies; here every rank WRITES its partial straight into a receive slot
// in each peer's memory (plain stores through the NVLink / NVSwitch peer mapping), raises a counter there, waits
// for the peers' counters in its own memory and adds the slots in rank order - one kernel, one link crossing, and
// every rank forms the sum in the same order, so the ranks' residual streams stay bit-identical.
//
// Memory of one rank: one allocation, the same layout on every rank (peer_layout.cuh), shared with the others
// through a CUDA IPC handle or - same process - by address.
// Two channels = the two module chains of a decode step (attention modules, MLP modules): each chain's exchanges are
// ordered on their own stream on every rank.  Two parities: a rank can start exchange t + 1 of a channel while a peer
// still adds the slots of exchange t, but it cannot start t + 2 before it has received that peer's part of t + 1,
// which the peer sends after it is done with t.
// Every wait is bounded (about 0.3 s): on expiry the kernel sets LADDER_DEV_TIMEOUT in the status word it was
// given, skips the sum and returns.  No multicast loads, no multimem: plain peer stores and local loads.
#include <cuda_runtime.h>
#include <stdint.h>

#include <string.h>

#include <new>

#include "../../include/ladder.h"
#include "common.cuh"
#include "peer_layout.cuh"

namespace {

using ladder::PeerView;
using Header = ladder::PeerHeader;
constexpr int kMaxWorld = LADDER_PEER_MAX_WORLD;
static_assert(kMaxWorld == ladder::kPeerMaxWorld, "world limit");
constexpr int kCtas = 16;       // CTAs per exchange kernel: the same on every rank (the counters count them)
constexpr int kThreads = 512;
constexpr long long kWaitCycles = 600000000ll;  // bound of a wait: ~0.3 s at 1.9 GHz
constexpr size_t kHeaderBytes = ladder::kPeerHeaderBytes;
using PeerArgs = PeerView;

__device__ __forceinline__ float* slot(unsigned char* base, const PeerArgs& a, int channel, int parity, int from) {
  return ladder::peer_slot(base, a.world, a.max_floats, channel, parity, from);
}
__device__ __forceinline__ uint32_t ld_acquire_sys(const uint32_t* p) { return ladder::peer_ld_acquire_sys(p); }
__device__ __forceinline__ void red_release_sys_add(uint32_t* p, uint32_t v) { ladder::peer_red_release_sys_add(p, v); }

// partial[0 .. count) += the other ranks' partials (in place, rank order).  count a multiple of 4.
__global__ void __launch_bounds__(kThreads) peer_all_reduce_kernel(PeerArgs a, int channel, float* partial, int64_t count,
                                                                   int32_t* status) {
  __shared__ int timed_out;
  Header* mine = reinterpret_cast<Header*>(a.base[a.rank]);
  const uint32_t turn = *reinterpret_cast<volatile uint32_t*>(&mine->turn[channel]);
  const int parity = turn & 1;
  const int64_t n4 = count >> 2;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  const int64_t first = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (threadIdx.x == 0) timed_out = 0;

  // 1. push: my partial into slot [channel][parity][my rank] of every rank (my own included), peers first
  const float4* src = reinterpret_cast<const float4*>(partial);
  for (int o = 1; o <= a.world; ++o) {
    const int p = (a.rank + o) % a.world;
    float4* dst = reinterpret_cast<float4*>(slot(a.base[p], a, channel, parity, a.rank));
    for (int64_t i = first; i < n4; i += stride) dst[i] = src[i];
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence_system();  // the CTA's stores (ordered before this thread by the barrier) before the counters
    for (int o = 1; o <= a.world; ++o) {
      const int p = (a.rank + o) % a.world;
      red_release_sys_add(&reinterpret_cast<Header*>(a.base[p])->arrive[channel][a.rank], 1u);
    }
  }

  // 2. wait until every rank's kCtas CTAs of this exchange have arrived here
  if (threadIdx.x < a.world) {
    const uint32_t target = (turn + 1u) * static_cast<uint32_t>(gridDim.x);
    const uint32_t* c = &mine->arrive[channel][threadIdx.x];
    bool ok = static_cast<int32_t>(ld_acquire_sys(c) - target) >= 0;
    if (!ok) {
      // Poll without sleeping, bounded by the SM's cycle counter (about 0.3 s).
      const long long t0 = clock64();
      for (uint32_t i = 1; !ok; ++i) {
        ok = static_cast<int32_t>(ld_acquire_sys(c) - target) >= 0;
        if (!ok && (i & 255u) == 0 && clock64() - t0 > kWaitCycles) break;
      }
    }
    if (!ok) {
      timed_out = 1;
      if (status) atomicOr(status, LADDER_DEV_TIMEOUT);
    }
  }
  __syncthreads();

  // 3. sum the slots in rank order (the same order on every rank)
  if (!timed_out) {
    float4* out = reinterpret_cast<float4*>(partial);
    for (int64_t i = first; i < n4; i += stride) {
      float4 s = __ldcg(reinterpret_cast<const float4*>(slot(a.base[a.rank], a, channel, parity, 0)) + i);
      for (int r = 1; r < a.world; ++r) {
        const float4 v = __ldcg(reinterpret_cast<const float4*>(slot(a.base[a.rank], a, channel, parity, r)) + i);
        s.x += v.x, s.y += v.y, s.z += v.z, s.w += v.w;
      }
      out[i] = s;
    }
  }

  // 4. the last CTA to finish moves the channel on (also after a time-out: the counters stay in step)
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    if (atomicAdd(&mine->ticket[channel], 1u) == gridDim.x - 1) {
      mine->ticket[channel] = 0;
      mine->turn[channel] = turn + 1u;
      __threadfence();
    }
  }
}

}  // namespace

struct ladder_peer {
  int world = 0, rank = 0;
  size_t max_floats = 0, bytes = 0;
  unsigned char* base[kMaxWorld] = {};
  bool ipc[kMaxWorld] = {};  // mapped with cudaIpcOpenMemHandle (to be closed)
};

namespace {
bool connected(const ladder_peer* p) {
  for (int r = 0; r < p->world; ++r)
    if (!p->base[r]) return false;
  return true;
}
Header* header(const ladder_peer* p, int r) { return reinterpret_cast<Header*>(p->base[r]); }
}  // namespace

namespace ladder {
bool peer_view(const ladder_peer* p, PeerView* out) {
  if (!p || !connected(p)) return false;
  for (int r = 0; r < kPeerMaxWorld; ++r) out->base[r] = r < p->world ? p->base[r] : nullptr;
  out->world = p->world;
  out->rank = p->rank;
  out->max_floats = p->max_floats;
  return true;
}
}  // namespace ladder

extern "C" {

ladder_status_t ladder_peer_create(int32_t world, int32_t rank, int64_t max_floats, ladder_peer_t** out) {
  if (!out || world < 1 || world > kMaxWorld || rank < 0 || rank >= world || max_floats < 4 || (max_floats & 3))
    return LADDER_ERR_INVALID_ARG;
  *out = nullptr;
  ladder_peer* p = new (std::nothrow) ladder_peer();
  if (!p) return LADDER_ERR_OOM;
  p->world = world;
  p->rank = rank;
  p->max_floats = static_cast<size_t>(max_floats);
  p->bytes = kHeaderBytes + sizeof(float) * 2 * 2 * world * 2 * p->max_floats;
  void* mem = nullptr;
  if (cudaMalloc(&mem, p->bytes) != cudaSuccess) {
    cudaGetLastError();
    delete p;
    return LADDER_ERR_OOM;
  }
  if (cudaMemset(mem, 0, p->bytes) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
    cudaFree(mem);
    delete p;
    return LADDER_ERR_CUDA;
  }
  p->base[rank] = static_cast<unsigned char*>(mem);
  *out = p;
  return LADDER_OK;
}

ladder_status_t ladder_peer_export(const ladder_peer_t* p, void* handle) {
  if (!p || !handle) return LADDER_ERR_INVALID_ARG;
  static_assert(sizeof(cudaIpcMemHandle_t) == LADDER_PEER_HANDLE_BYTES, "IPC handle size");
  return cudaIpcGetMemHandle(static_cast<cudaIpcMemHandle_t*>(handle), p->base[p->rank]) == cudaSuccess ? LADDER_OK
                                                                                                          : LADDER_ERR_CUDA;
}

void* ladder_peer_local_base(const ladder_peer_t* p) { return p ? p->base[p->rank] : nullptr; }

ladder_status_t ladder_peer_connect(ladder_peer_t* p, int32_t r, const void* ipc_handle, void* same_process_base) {
  if (!p || r < 0 || r >= p->world || r == p->rank || p->base[r] || (ipc_handle != nullptr) == (same_process_base != nullptr))
    return LADDER_ERR_INVALID_ARG;
  if (same_process_base) {
    p->base[r] = static_cast<unsigned char*>(same_process_base);
    return LADDER_OK;
  }
  void* mapped = nullptr;
  cudaIpcMemHandle_t h;
  memcpy(&h, ipc_handle, sizeof(h));
  if (cudaIpcOpenMemHandle(&mapped, h, cudaIpcMemLazyEnablePeerAccess) != cudaSuccess) {
    cudaGetLastError();
    return LADDER_ERR_CUDA;
  }
  p->base[r] = static_cast<unsigned char*>(mapped);
  p->ipc[r] = true;
  return LADDER_OK;
}

int32_t ladder_peer_connected(const ladder_peer_t* p) { return (p && connected(p)) ? 1 : 0; }
int32_t ladder_peer_world(const ladder_peer_t* p) { return p ? p->world : 0; }
int32_t ladder_peer_rank(const ladder_peer_t* p) { return p ? p->rank : -1; }
int64_t ladder_peer_max_floats(const ladder_peer_t* p) { return p ? static_cast<int64_t>(p->max_floats) : 0; }
int32_t ladder_peer_ctas_per_exchange(void) { return kCtas; }

ladder_status_t ladder_peer_destroy(ladder_peer_t* p) {
  if (!p) return LADDER_OK;
  for (int r = 0; r < p->world; ++r)
    if (p->ipc[r] && p->base[r]) cudaIpcCloseMemHandle(p->base[r]);
  if (p->base[p->rank]) cudaFree(p->base[p->rank]);
  delete p;
  return LADDER_OK;
}

ladder_status_t ladder_peer_all_reduce_sum(ladder_peer_t* p, int32_t channel, float* partial, int64_t count,
                                           int32_t* device_status, void* cuda_stream) {
  if (!p || !partial || channel < 0 || channel > 1 || count < 0 || (count & 3) ||
      static_cast<size_t>(count) > p->max_floats || (reinterpret_cast<uintptr_t>(partial) & 15))
    return LADDER_ERR_INVALID_ARG;
  if (!connected(p)) return LADDER_ERR_STATE;
  if (count == 0) return LADDER_OK;
  PeerArgs a = {};
  ladder::peer_view(p, &a);
  peer_all_reduce_kernel<<<kCtas, kThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(a, channel, partial, count,
                                                                                        device_status);
  return cudaGetLastError() == cudaSuccess ? LADDER_OK : LADDER_ERR_CUDA;
}

// Connectivity check (host copies, no kernel): write `value` into this rank's probe word in rank r's memory /
// read the word rank `from` has written here.
ladder_status_t ladder_peer_probe_write(ladder_peer_t* p, int32_t r, uint32_t value) {
  if (!p || r < 0 || r >= p->world || !p->base[r]) return LADDER_ERR_INVALID_ARG;
  // a copy from pageable memory may return before the DMA has reached the destination: wait for it, the reader
  // is another process and only a host-side barrier orders it after this call
  return (cudaMemcpy(&header(p, r)->probe[p->rank], &value, sizeof(value), cudaMemcpyHostToDevice) == cudaSuccess &&
          cudaDeviceSynchronize() == cudaSuccess)
             ? LADDER_OK
             : LADDER_ERR_CUDA;
}
ladder_status_t ladder_peer_probe_read(const ladder_peer_t* p, int32_t from, uint32_t* value) {
  if (!p || !value || from < 0 || from >= p->world) return LADDER_ERR_INVALID_ARG;
  return cudaMemcpy(value, &header(p, p->rank)->probe[from], sizeof(*value), cudaMemcpyDeviceToHost) == cudaSuccess
             ? LADDER_OK
             : LADDER_ERR_CUDA;
}

// For tests that play a missing rank on the same GPU: where rank `from`'s data of (channel, parity) lands in this
// rank's memory, and the counter that says it has.
float* ladder_peer_slot(const ladder_peer_t* p, int32_t channel, int32_t parity, int32_t from) {
  if (!p || channel < 0 || channel > 1 || parity < 0 || parity > 1 || from < 0 || from >= p->world) return nullptr;
  return ladder::peer_slot(p->base[p->rank], p->world, p->max_floats, channel, parity, from);
}
uint32_t* ladder_peer_counter(const ladder_peer_t* p, int32_t channel, int32_t from) {
  if (!p || channel < 0 || channel > 1 || from < 0 || from >= p->world) return nullptr;
  return &header(p, p->rank)->arrive[channel][from];
}

}  // extern "C"
