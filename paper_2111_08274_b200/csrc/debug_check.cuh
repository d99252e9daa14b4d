// Bounds checks of the debug build (-DHADFL_DEBUG, libhadfl_debug.so).
//
// In that build every access the kernels make to the parameter and momentum arenas and every
// store to the library's scratch buffers is first checked against a table of device address
// ranges that the host registers (arenas, scratch, staging row).  An access that is not wholly
// inside one of them is SKIPPED (a load returns zeros, a store stores nothing) and recorded in an
// error word with the offending address; the kernel carries on and ends normally - no trap, no
// assert - and the next synchronising call of the library returns HADFL_ERR_STATE.  This is the
// stand-in for a memory checker where none can be run.  In the normal build access_ok is a
// constant `true` and the checks vanish.
#pragma once
#include <stdint.h>

#include "philox.cuh"  // HADFL_HD

namespace hadfl {

// [addr, addr + nbytes) lies inside [lo, hi)?  Written so that nothing overflows.
HADFL_HD bool range_holds(uint64_t lo, uint64_t hi, uint64_t addr, uint64_t nbytes) {
  return lo <= hi && addr >= lo && addr <= hi && nbytes <= hi - addr;
}

constexpr int kDebugRanges = 64;

struct DebugRanges {
  uint64_t lo[kDebugRanges], hi[kDebugRanges];
  int32_t n;
  // written by kernels only:
  uint32_t error;     // 0 = every access so far was in range
  uint64_t bad_addr;  // first address that was not
};

#if defined(HADFL_DEBUG) && defined(__CUDACC__)
__device__ DebugRanges g_debug;

__device__ __forceinline__ bool access_ok(const void *p, size_t nbytes) {
  if (nbytes == 0) return true;  // nothing is touched (lanes beyond the end of a row)
  const uint64_t a = (uint64_t)(uintptr_t)p;
  const int n = g_debug.n;
  for (int r = 0; r < n; ++r)
    if (range_holds(g_debug.lo[r], g_debug.hi[r], a, (uint64_t)nbytes)) return true;
  if (atomicExch(&g_debug.error, 1u) == 0u) g_debug.bad_addr = a;
  return false;
}
#elif defined(__CUDACC__)
__device__ __forceinline__ constexpr bool access_ok(const void *, size_t) { return true; }
#endif

}  // namespace hadfl
