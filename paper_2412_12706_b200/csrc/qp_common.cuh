// Shared device helpers and launch-side declarations of the quantized-pruning kernels.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/qp.h"

namespace qp {

using bf16 = __nv_bfloat16;

__device__ __forceinline__ float bf16_bits_to_f32(uint16_t h) { return __uint_as_float((uint32_t)h << 16); }
__device__ __forceinline__ float bf16lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

// D(16x8,f32) += A(16x16,bf16,row) * B(16x8,bf16,col)
__device__ __forceinline__ void mma_bf16_m16n8k16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// D(16x8,f32) += A(16x16,f16,row) * B(16x8,f16,col)
__device__ __forceinline__ void mma_f16_m16n8k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                 uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t saddr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(saddr));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3,
                                                  uint32_t saddr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(saddr));
}

__device__ __forceinline__ void cp_async16(uint32_t saddr, const void* gptr) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(saddr), "l"(gptr));
}
// Kernels of a chain that are launched with launch_chained() begin with chain_enter(): the next kernel of the stream
// may be launched at once (its blocks become resident as this grid's last blocks have started), and this grid waits
// until the previous kernel of the stream has completed and its writes are visible before it touches memory.  Only the
// launch latency overlaps; every data dependence is a full kernel boundary as before.
__device__ __forceinline__ void chain_enter() {
  asm volatile("griddepcontrol.launch_dependents;\n" ::);
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

// ---- launch-side entry points (one per .cu file) --------------------------------------------

struct ScoreDims {
  int Bt, Hq, Hkv, D, L, w, pool;
};
// workspace carving for S1 (all offsets 256-byte aligned)
struct ScoreWorkspace {
  size_t stat_partial, rowstat, votes_partial, pooled, error, total;   // error: one int, the last 256 bytes
  int n_rb, n_tiles, n_vote_tiles;
};
ScoreWorkspace score_workspace(int Bt, int Hq, int Hkv, int L, int w);
cudaError_t launch_window_scores(const void* Qwin, const void* K, const ScoreDims& d, float* scores, void* ws,
                                 cudaStream_t st);
// The same for n_layers layers of one shape in one sequence of launches: the layers are stacked along the batch
// dimension of the scratch arrays (ws: score_workspace(Bt * n_layers, ...)) and of scores [n_layers, Bt, Hkv, P].
cudaError_t launch_window_scores_layers(int n_layers, const void* const* Qwin, const void* const* K, const ScoreDims& d,
                                        float* scores, void* ws, cudaStream_t st);
// per-layer inputs of the score sweeps, passed by value
template <int NL>
struct ScorePtrs {
  const bf16* q[NL];
  const bf16* k[NL];
};

// tcgen05 / TMEM form of the two score sweeps (same outputs as score_sweep_kernel)
bool score_tc_supported(int D);
cudaError_t launch_score_sweep_tc(int pass, int n_layers, const void* const* q, const void* const* k, const ScoreDims& d,
                                  const ScoreWorkspace& s, float scale_log2, float2* stat_partial, const float2* rowstat,
                                  float* votes_partial, int* error_word, cudaStream_t st, int bh0, int bh_count,
                                  int* n_splits, int n_stat = 0);

cudaError_t launch_select_topk(const float* scores, int BH, int L, int w, int n_keep, int32_t* kept, cudaStream_t st);
// n_layers layers in one launch: scores [n_layers, BH, P]; kept[l] int32 [BH, n_keep[l]]
cudaError_t launch_select_topk_layers(int n_layers, const float* scores, int BH, int L, int w, const int* n_keep,
                                      int32_t* const* kept, cudaStream_t st);

// per-head token counts under a shared layer budget; kept_flat: scratch int32 [Bt, min(Hkv*(n_mean-w), Hkv*P) + 1]
cudaError_t launch_head_budgets(const float* scores, int Bt, int Hkv, int L, int w, int n_mean, int unit,
                                int32_t* n_heads, int32_t* kept_flat, cudaStream_t st);

cudaError_t launch_gather_quantize(const void* K, const void* V, const int32_t* kept, int L, const qp_cache& c,
                                   cudaStream_t st);
// n_layers caches of one shape (n_keep may differ) in one launch; kept[l] int32 [BH, caches[l].n_keep]
cudaError_t launch_gather_quantize_layers(int n_layers, const void* const* K, const void* const* V,
                                          const int32_t* const* kept, int L, const qp_cache* caches, cudaStream_t st);
// tokens per (batch, KV head) the arrays of c are sized for
inline int cache_capacity(const qp_cache& c) { return c.n_cap > 0 ? c.n_cap : c.n_keep; }

// decode-time appends: new rows into the tail (or, at 16 bit, into the cache), and the quantization of full
// tails into the caches' next group; each one launch over all layers
cudaError_t launch_append_rows(int n_layers, const void* const* k_new, const void* const* v_new, const qp_cache* caches,
                               const qp_tail* tails, cudaStream_t st);
cudaError_t launch_flush_tails(int n_layers, const int* which, const qp_cache* caches, const qp_tail* tails,
                               cudaStream_t st);

// The other quantization strategies (qp_strategy): key grouping axis and outlier side lists, device pointers.
struct SideList {
  const int32_t* idx;       // [BH, cap] ascending t*D + d
  const uint16_t* val;      // [BH, cap] bf16
  const int32_t* cnt;       // [BH]
  const int32_t* tile_ptr;  // [BH, n_tiles + 1]: entries of tokens 32i .. 32i+31 are [tile_ptr[i], tile_ptr[i+1])
  int cap, n_tiles;
};
struct DecEx {
  int k_axis;               // 0: key groups per channel over g tokens; 1: per token over g channels
  int has_side;
  SideList k, v;
};
cudaError_t launch_gather_quantize_ex(const void* K, const void* V, const int32_t* kept, int L, const qp_cache& c,
                                      const qp_strategy& s, cudaStream_t st);
cudaError_t launch_decode_ex(const struct DecTable& tab, const struct DecDims& d, const DecEx& ex, void* workspace,
                             cudaStream_t st);

// decode: per-layer device pointers, passed by value as a kernel parameter
struct DecLayer {
  const void* kc;
  const void* vc;
  const __half* ks;
  const __half* kz;
  const __half* vs;
  const __half* vz;
  const void* q;
  void* out;
  int n;          // kept tokens of this layer
  int part_base;  // chunked kernel: first partial slot of this layer (in units of (bh, split) slots)
  int tile_base;  // flat-range kernel: index of this layer's first 32-token tile in the flat tile sequence
  int ns;         // tokens the arrays have room for per (batch, KV head): the stride between heads (>= n)
};
struct DecTable {
  int n_layers;
  int chunk;        // chunked kernel: tokens per split
  int total_tiles;  // flat-range kernel: tiles of all layers and heads
  int n_workers;    // flat-range kernel: workers (blocks or warps, by kernel), each owning total_tiles / n_workers consecutive tiles
  int paired;       // flat-range kernel: 1 = planned for a stream on which consecutive calls overlap (see decode_plan)
  int wide;         // flat-range kernel: 1 = the build with more resident workers per SM (long ranges), see decode_plan
  DecLayer l[QP_MAX_LAYERS];
};
struct DecDims {
  int Bt, Hq, Hkv, D, bits, group;
};
// unquantized tail tokens of each layer (bf16 [Bt,Hkv,group,D]); read by the merge step only
struct TailLayer {
  const void* kt;
  const void* vt;
  int n_tail, pad_;
};
struct TailTable {
  TailLayer l[QP_MAX_LAYERS];
};
#ifndef QP_MAX_DECODE_WORKERS
#define QP_MAX_DECODE_WORKERS 2432
#endif
constexpr int kMaxDecodeWorkers = QP_MAX_DECODE_WORKERS;
// Chooses the decomposition for the layers in tab (n and pointers already set), fills chunk / part_base or
// tile_base / total_tiles / n_workers and returns the bytes of partial records the launch needs.
// paired: the stream lets consecutive calls overlap (two calls share the GPU most of the time), so a small launch
// does better with fewer, longer-lived workers; alone on the GPU it wants as many as it can feed.
size_t decode_plan(DecTable& tab, const DecDims& d, bool paired);
size_t decode_plan_chunked(DecTable& tab, const DecDims& d);
// the flat-range decomposition for a kernel with `workers_per_sm` resident workers; returns the bytes of ONE record area
size_t decode_plan_flat(DecTable& tab, const DecDims& d, int workers_per_sm, int tiles_per_worker_min);   // the chunked decomposition, whatever the shape
// Upper bound of decode_plan's result for one layer of n_keep tokens, whatever else is in the launch.
size_t decode_workspace_bound(const DecDims& d, int n_keep);
// Workspace of the tensor-core kernels: two areas of partial records, used by alternate calls (parity), so that
// a call's attention kernel can write its records while the previous call's merge kernel still reads its own.
struct DecWorkspace {
  size_t record_bytes;   // of one area, a multiple of 256
  size_t total_bytes() const { return 2 * record_bytes; }
};
DecWorkspace decode_workspace_layout(const DecTable& tab, const DecDims& d);
// parity: which half this call uses.  overlap_prev: the attention kernel may start while the stream's previous
// kernel (an earlier decode call) still runs; the caller guarantees that this launch reads nothing that kernel
// writes and that the earlier call used the other half.
// tails: null, or the layers' tails (the merge step then adds their tokens to the softmax)
cudaError_t launch_decode(const DecTable& tab, const DecDims& d, void* workspace, int parity, cudaStream_t st,
                          bool overlap_prev, const TailTable* tails = nullptr);
// merge of the partial records plus the tail tokens, for either decomposition (chunked: tab.n_workers == 0)
cudaError_t launch_merge_tail(const DecTable& tab, const DecDims& d, const float* partials, const TailTable& tails,
                              cudaStream_t st, bool programmatic);
int sm_count();   // SMs of the current device (cached)
// tensor-core split-K kernel and its merge
bool decode_mma_supported(const DecDims& d);
int decode_mma_workers_per_sm(const DecDims& d);     // workers (see DecTable::n_workers) resident per SM
int decode_mma_tiles_per_worker_min(const DecDims& d, long long total_tiles, bool paired);   // small launches: fewer workers, not emptier ones
int decode_mma_wide_workers_per_sm(const DecDims& d, int* min_tiles);
cudaError_t launch_decode_mma(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st,
                              bool overlap_prev, const TailTable* tails = nullptr);

}  // namespace qp
