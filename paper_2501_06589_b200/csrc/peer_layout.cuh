// Layout of one rank's peer-exchange memory (the same on every rank) and how kernels address it.
//   header (1 KiB):
//     arrive[channel][rank]  uint32, CTA arrivals of `rank`'s data on this channel in THIS rank's memory (monotonic)
//     turn[channel]          uint32, exchanges this rank has consumed on the channel (receive-slot parity = turn & 1)
//     ticket[channel]        uint32, CTAs of the consuming kernel that are done (the last one advances `turn`)
//     probe[rank]            uint32, connectivity check (host copies only)
//   rx[channel][parity][rank][2 * max_floats]  the receive slots: max_floats (value, sequence number) pairs when the
//                          exchange is fused into a model's kernels, max_floats plain values (first half) for the
//                          stand-alone kernel
#pragma once
#include <stddef.h>
#include <stdint.h>

namespace ladder {

constexpr int kPeerMaxWorld = 8;
constexpr size_t kPeerHeaderBytes = 1024;

struct PeerHeader {
  uint32_t arrive[2][kPeerMaxWorld];
  uint32_t turn[2];
  uint32_t ticket[2];
  uint32_t probe[kPeerMaxWorld];
};
static_assert(sizeof(PeerHeader) <= kPeerHeaderBytes, "header size");

// Every rank's block as seen from this device (base[rank] = the local one).  world == 0: no peer exchange.
struct PeerView {
  unsigned char* base[kPeerMaxWorld];
  int world, rank;
  size_t max_floats;
};

__host__ __device__ inline float* peer_slot(unsigned char* base, int world, size_t max_floats, int channel, int parity,
                                            int from) {
  return reinterpret_cast<float*>(base + kPeerHeaderBytes) +
         ((static_cast<size_t>(channel) * 2 + parity) * world + from) * (2 * max_floats);
}
__host__ __device__ inline PeerHeader* peer_header(unsigned char* base) { return reinterpret_cast<PeerHeader*>(base); }

#ifdef __CUDACC__
// Counting an arrival after the data (the caller has run __threadfence_system() after its stores) and reading the
// counters before the data: the stand-alone exchange kernel.
__device__ __forceinline__ uint32_t peer_ld_acquire_sys(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void peer_red_release_sys_add(uint32_t* p, uint32_t v) {
  asm volatile("red.release.sys.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// The fused exchange writes every value together with the sequence number of its exchange as ONE aligned 8-byte
// store, and the reader polls the pair until the number is the one it expects: no counters, no fences, one link
// crossing (the technique of NCCL's low-latency protocol; it rests on aligned 8-byte stores arriving whole).
__device__ __forceinline__ void peer_st_pair(uint2* p, float value, uint32_t seq) {
  asm volatile("st.relaxed.sys.global.v2.u32 [%0], {%1, %2};" ::"l"(p), "r"(__float_as_uint(value)), "r"(seq) : "memory");
}
__device__ __forceinline__ uint4 peer_ld_pairs(const uint4* p) {  // two pairs: (x, y) and (z, w)
  uint4 v;
  asm volatile("ld.relaxed.sys.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}
#endif

}  // namespace ladder
