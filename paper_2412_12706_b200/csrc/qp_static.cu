// qp_decode_attn_static: decode attention for callers that cannot allocate device memory.
//
// The split-K decode kernels need scratch for the per-split partial results.  The other
// entry points take that scratch from the caller; this one keeps it in a fixed array that is
// part of the library image, so the caller passes only inputs and outputs.
#include <algorithm>
#include <atomic>

#include "qp_common.cuh"

namespace {

// Scratch shared by every call on a device.  It lives in each GPU's memory from the moment the
// library is loaded on that GPU until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[QP_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
// Device address of g_static_scratch per CUDA device.  The array's name is only a host-side
// handle in host code; the address a kernel can use must be asked for, with that device current.
// Filled on the first call on each device; host threads that race on a first call all store the same value.
std::atomic<void*> g_scratch_addr[kMaxDevices] = {};

qp_status static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return QP_ERR_CUDA;
  void* p = g_scratch_addr[dev].load(std::memory_order_acquire);
  if (!p) {
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return QP_ERR_CUDA;
    g_scratch_addr[dev].store(p, std::memory_order_release);
  }
  *out = p;
  return QP_OK;
}

}  // namespace

extern "C" qp_status qp_decode_attn_static(const void* q, const qp_cache* cache, void* out, void* stream) {
  if (!cache) return QP_ERR_INVALID_ARG;
  // Scratch this cache needs: (max, sum, acc[D]) records, one per query head of the group for every
  // (batch, KV head, token split) the decode launch will use for this much work.
  const size_t coarse = qp_decode_workspace_bytes(cache);
  if (coarse == 0) return QP_ERR_INVALID_ARG;   // invalid descriptor
  const qp::DecDims d{cache->batch, cache->n_q_heads, cache->n_kv_heads, cache->head_dim, cache->bits, cache->group};
  qp::DecTable plan;
  plan.n_layers = 1;
  plan.l[0].n = cache->n_keep;
  // the plans qp_decode_attn may make for this cache (it depends on the stream's overlap setting)
  const size_t need = std::max(qp::decode_plan(plan, d, false), qp::decode_plan(plan, d, true));
  if (need > (size_t)QP_STATIC_SCRATCH_BYTES) return QP_ERR_WORKSPACE;
  void* scratch = nullptr;
  const qp_status s = static_scratch(&scratch);
  if (s != QP_OK) return s;
  // Every partial record that the merge reads is written first by the attention kernel of the same
  // call, so nothing in the array has to start at zero.
  return qp_decode_attn(q, cache, out, scratch, QP_STATIC_SCRATCH_BYTES, stream);
}
