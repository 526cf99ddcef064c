// Device helpers shared by the tensor-core decode kernels.
#pragma once

#include "qp_common.cuh"

namespace qp {

__device__ __forceinline__ uint32_t hmul2_u32(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("mul.rn.f16x2 %0, %1, %2;\n" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ uint4 lds128(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];\n" : "=r"(v.x), "=r"(v.y) : "r"(a));
  return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];\n" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts64(uint32_t a, uint32_t x, uint32_t y) {
  asm volatile("st.shared.v2.u32 [%0], {%1,%2};\n" ::"r"(a), "r"(x), "r"(y));
}

// 2^x for x <= 0 (softmax weights): the hardware approximation, about 2 ulp, flushes tiny results to 0
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

// Order of consecutive decode calls on one stream when they are allowed to overlap (programmatic dependent
// launch).  Kernels of a stream: A_N (attention of call N), M_N (its merge), optionally P (rows of an appended
// token), A_{N+1}, ...  Every kernel executes griddepcontrol.wait before it ends, so "X has ended" implies
// "everything before X has ended".  The merge and append kernels pass the launch permission on as soon as they
// start; an attention kernel passes it on only AFTER its own wait has returned (pdl_gate), a few tiles before
// its range ends.  So A_{N+1} can begin only when some thread of A_N is past its wait, i.e. when the kernel
// before A_N (M_{N-1}, or an append after it) and with it everything of call N-1 and earlier has ended:
// at most A_N, M_N (and an append) and A_{N+1} are in flight together, however small the grids are.  A_{N+1}
// therefore needs to be checked only against call N (the host does: it reads none of call N's outputs) and
// writes the workspace half that call N-1, which has ended, used.
__device__ __forceinline__ void pdl_gate() {
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
}
// the gate sits this many tiles before the end of a worker's range (or at its start, for shorter ranges): late
// enough that the previous call's merge has normally ended by then, early enough to hide the next launches
#ifndef QP_GATE_TILES
#define QP_GATE_TILES 2
#endif
#ifndef QP_GATE_EIGHTHS
#define QP_GATE_EIGHTHS 4
#endif
constexpr int kGateTiles = QP_GATE_TILES;
// first tile a worker computes AFTER its gate, for a range of `total` tiles
__device__ __forceinline__ int gate_tile(int total) {
  const int lead = max(kGateTiles, (total * QP_GATE_EIGHTHS) >> 3);
  return total > lead ? total - lead : 0;
}

// Work decomposition ("stream-K" over tokens): the 32-token tiles of all (layer, batch, KV head)
// triples form one flat sequence of T tiles; block w of W owns the contiguous range
// [w*T/W, (w+1)*T/W), so every block streams the same number of bytes (+-1 tile), the grid is one
// wave of resident blocks and a block pays its pipeline ramp once.  A range that crosses a head
// boundary is processed head by head ("segments"); each (head, block) pair that meets leaves one
// partial record at slot head + block (heads and blocks both advance monotonically along the flat
// sequence, so head + block is unique), which the merge kernel finds again by the same arithmetic.
struct SkOwner {
  long long T, W;
  __host__ __device__ long long start(long long w) const { return w * T / W; }
  // the block whose range holds flat tile f is ((f + 1) * W - 1) / T
};


// Launches an attention kernel; with overlap_prev as a programmatic dependent of the stream's previous kernel
// (it may start while that one still runs; see launch_decode).
template <typename K>
cudaError_t launch_attention(K kernel, int blocks, int threads, size_t smem, cudaStream_t st, bool overlap_prev,
                             const DecTable& tab, const DecDims& d, float* partials) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks);
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = overlap_prev ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, tab, d, partials);
}

// launchers of the per-bit-width attention kernels
cudaError_t launch_decode_mma4(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st,
                               bool overlap_prev);
cudaError_t launch_decode_mma2(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st, bool overlap_prev);
bool decode_mma2_supported(const DecDims& d);
int decode_mma2_workers_per_sm();
cudaError_t launch_decode_mma8(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st, bool overlap_prev);
int decode_mma8_blocks_per_sm();
int decode_mma8_warps();
cudaError_t launch_decode_mma16(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st, bool overlap_prev);
// 4-bit caches whose keys are quantized token by token (qp_strategy.k_axis = 1): attention kernel only
bool decode_mma4t_supported(const DecDims& d);
int decode_mma4t_workers_per_sm();
cudaError_t launch_decode_mma4t(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st);
// the merge kernels of the flat-range decomposition (records of every attention kernel above)
cudaError_t launch_merge_flat(const DecTable& tab, const DecDims& d, const float* partials, cudaStream_t st);
int decode_mma16_blocks_per_sm();

// opt in to more than 48 KB of dynamic shared memory, once per device and kernel
template <typename K>
cudaError_t allow_smem(K kernel, size_t bytes, unsigned char (&done)[64]) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (done[dev]) return cudaSuccess;
  const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess) done[dev] = 1;
  return e;
}

}  // namespace qp
