// State words and the bounded wait of the decoupled look-back scans (selection offsets, digit offsets of the
// ranking passes, block offsets of the unframed stream).  A state word carries a 62-bit value under two flag bits;
// a block publishes its own aggregate first and its inclusive prefix once it knows it, and walks back over its
// predecessors until it meets a prefix.  Every wait is bounded: after kMaxPolls polls it gives up, reports
// DEVICE_TIMEOUT and the kernel carries on to its end with void results.
#pragma once

#include "cvlc_common.cuh"

namespace cvlc {

#ifdef __CUDACC__

constexpr unsigned long long kFlagAgg = 1ull << 62;     // tile aggregate published
constexpr unsigned long long kFlagPrefix = 2ull << 62;  // inclusive prefix published
constexpr unsigned long long kFlagMask = 3ull << 62;
constexpr unsigned long long kValMask = ~kFlagMask;
constexpr int kMaxPolls = 1 << 20;  // bounded wait of the look-back; then DEVICE_TIMEOUT

__device__ __forceinline__ unsigned long long ld_relaxed(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed(unsigned long long* p, unsigned long long v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// Waits (bounded) until a look-back state word carries a flag.  Returns 0 after a timeout.
__device__ __forceinline__ unsigned long long wait_state(const unsigned long long* p, int32_t* status, int max_polls = kMaxPolls) {
  unsigned long long v = ld_relaxed(p);
  int polls = 0;
  while ((v & kFlagMask) == 0) {
    if (++polls > max_polls) {
      set_status(status, CVLC_ERR_DEVICE_TIMEOUT);
      return 0;
    }
    if (polls > 64) __nanosleep(64);
    v = ld_relaxed(p);
  }
  return v;
}


#endif  // __CUDACC__

}  // namespace cvlc
