// Debug build with device-side range checks (compile with -DQP_CHECKED; the build script makes it as
// libqp_checked.so).  Every index that a kernel takes from DEVICE memory before using it as an address (the kept
// positions, the side lists' entries and tile pointers; also the output positions the top-k kernels compute from their counts) is compared with its limit first.  A violation never traps:
// the first one is recorded (site, index, limit), all are counted, and the access is redirected to element 0 or
// skipped.  The host reads the record with qp_debug_check().  The normal build compiles the checks away.
#pragma once

#include <cuda_runtime.h>

#ifdef QP_CHECKED
namespace qp {
namespace checked {
// one copy per translation unit; qp_debug_check() collects them
static __device__ unsigned int g_word[4];   // 1 + site of the first violation, its index, its limit, violations
__device__ __forceinline__ bool in_range(long long idx, long long limit, unsigned site) {
  if (idx >= 0 && idx < limit) return true;
  if (atomicCAS(&g_word[0], 0u, site + 1u) == 0u) {
    g_word[1] = (unsigned)idx;
    g_word[2] = (unsigned)limit;
  }
  atomicAdd(&g_word[3], 1u);
  return false;
}
// reads and clears this translation unit's record (synchronises the device)
inline cudaError_t read_and_clear(unsigned int (&out)[4]) {
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return e;
  e = cudaMemcpyFromSymbol(out, g_word, sizeof(out));
  if (e != cudaSuccess) return e;
  const unsigned int zero[4] = {0u, 0u, 0u, 0u};
  return cudaMemcpyToSymbol(g_word, zero, sizeof(zero));
}
}  // namespace checked
}  // namespace qp
#define QP_IN_RANGE(idx, limit, site) qp::checked::in_range((long long)(idx), (long long)(limit), (site))
#else
#define QP_IN_RANGE(idx, limit, site) true
#endif

// sites
#define QP_SITE_GATHER_KEPT 1u      // gather + quantize: a kept position >= L
#define QP_SITE_ROWS_KEPT 2u        // 16-bit row gather: a kept position >= L
#define QP_SITE_SIDE_KEPT 3u        // side-list build: a kept position >= L
#define QP_SITE_SIDE_PTR 4u         // decode: a side list's tile pointer outside [0, cap]
#define QP_SITE_SIDE_IDX 5u         // decode: a side-list entry outside the cache
#define QP_SITE_TOPK_OUT 6u         // top-k: an output position computed from the counts >= k
