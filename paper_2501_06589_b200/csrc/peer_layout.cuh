// Layout of one rank's peer-exchange memory (the same on every rank) and how kernels address it.
//   header (1 KiB):
//     arrive[channel][rank]  uint32, CTA arrivals of `rank`'s data on this channel in THIS rank's memory (monotonic)
//     turn[channel]          uint32, exchanges this rank has consumed on the channel (receive-slot parity = turn & 1)
//     ticket[channel]        uint32, CTAs of the consuming kernel that are done (the last one advances `turn`)
//     probe[rank]            uint32, connectivity check (host copies only)
//   rx[channel][parity][rank][max_floats]  the receive slots
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
         ((static_cast<size_t>(channel) * 2 + parity) * world + from) * max_floats;
}
__host__ __device__ inline PeerHeader* peer_header(unsigned char* base) { return reinterpret_cast<PeerHeader*>(base); }

#ifdef __CUDACC__
__device__ __forceinline__ uint32_t peer_ld_acquire_sys(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void peer_red_release_sys_add(uint32_t* p, uint32_t v) {
  asm volatile("red.release.sys.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
#endif

}  // namespace ladder
