// Shared host/device helpers of the bsp library (status handling, bf16 access, small reductions).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "bsp.h"

namespace bsp {

// Last CUDA error seen by this host thread inside the library.
int& last_cuda_error_ref();

inline int cuda_fail(cudaError_t e) {
  last_cuda_error_ref() = static_cast<int>(e);
  return BSP_ERR_CUDA;
}

#define BSP_CUDA_TRY(expr)                                  \
  do {                                                      \
    cudaError_t _e = (expr);                                \
    if (_e != cudaSuccess) return ::bsp::cuda_fail(_e);     \
  } while (0)

// Kernel launches report configuration errors through cudaGetLastError.
#define BSP_LAUNCH_CHECK()                                  \
  do {                                                      \
    cudaError_t _e = cudaGetLastError();                    \
    if (_e != cudaSuccess) return ::bsp::cuda_fail(_e);     \
  } while (0)

inline bool aligned_to(const void* p, size_t a) {
  return (reinterpret_cast<uintptr_t>(p) % a) == 0;
}
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Number of blocks / groups per block for a geometry; returns false when `block` does not divide.
inline bool geometry(int rows, int cols, int block, int orient, int* n_blocks, int* n_groups) {
  if (orient == BSP_ORIENT_C) {
    if (rows % block) return false;
    *n_blocks = rows / block;
    *n_groups = cols;
  } else {
    if (cols % block) return false;
    *n_blocks = cols / block;
    *n_groups = rows;
  }
  return true;
}

// Common argument screening for calls that take (W, rows, cols, ldw, block, orient).
inline int check_matrix_args(const void* W, int rows, int cols, int ldw, int block, int orient) {
  if (W == nullptr || rows <= 0 || cols <= 0 || block <= 0) return BSP_ERR_ARG;
  if (orient != BSP_ORIENT_C && orient != BSP_ORIENT_R) return BSP_ERR_ARG;
  if (!aligned_to(W, 2)) return BSP_ERR_ARG;
  if (ldw < cols) return BSP_ERR_SHAPE;
  int nb, ng;
  if (!geometry(rows, cols, block, orient, &nb, &ng)) return BSP_ERR_SHAPE;
  return BSP_OK;
}

// Workspace of the pack calls: [per-block counts][per-group flags][per-group float32 S], each
// region 256-byte aligned.  (The fused call keeps per-block penalty partials in the S region.)
struct WsLayout {
  size_t counts_off, keep_off, sumsq_off, total;
};
inline WsLayout ws_layout(int n_blocks, int n_groups) {
  WsLayout L;
  const size_t groups = static_cast<size_t>(n_blocks) * n_groups;
  L.counts_off = 0;
  L.keep_off = round_up(sizeof(int32_t) * (static_cast<size_t>(n_blocks) + 1), 256);
  L.sumsq_off = L.keep_off + round_up(groups, 256);
  L.total = L.sumsq_off + round_up(groups * sizeof(float), 256);
  return L;
}


// One matrix of a launch of the vectorised orientation-C kernels (bsp_fused.cu).  Null output
// pointers switch the matching work off.
struct FusedJob {
  const uint16_t* W;
  int rows, cols, ldw, n_blocks;
  float threshold;
  const float* threshold_dev;
  float* norms;
  const float* gamma_in;
  float* gamma_out;
  double* penalty;             // job total (written by stage 2 from `partial`, or by atomics in stage 1)
  double* partial;             // per-block penalty partial sums, or null: stage 1 adds into *penalty
  uint8_t* flags;              // per-group keep flags (null: stage 1 skips the keep decision)
  int32_t* counts;             // per-block kept counts
  int32_t* blk_ptr;
  int32_t* idx;
  uint16_t* vals;
  int64_t* kept_weights;
  uint16_t* plan;
};
constexpr int kFusedMaxJobs = 96;     // per launch; the job table travels as a kernel parameter (about 15 KB)
constexpr int kFusedMaxCols = 4096;     // stage 2 keeps 12 bytes of shared memory per column
constexpr int kFusedMaxBlocks = 1024;   // stage 2 sums the counts before its block directly
// Stage 1: sums of squares -> norms / gamma / penalty and/or keep flags + counts, one pass over W.
int fused_stage1(const FusedJob* jobs, int n_jobs, int block, float eps, int squared, cudaStream_t s);
// Stage 2: blk_ptr, index lists, packed tiles, penalty totals, optional execution layout.
int fused_stage2(const FusedJob* jobs, int n_jobs, int block, cudaStream_t s);
// Streaming one-pass kernel for batches of any size (bsp_fused_stream.cu); *used = false means nothing was launched.
int fused_stream(const FusedJob* jobs, int n_jobs, int block, float eps, int squared, int32_t* const* part_counts,
                 double* const* part_partial, cudaStream_t s, bool* used);
// Whether a matrix can go through the vectorised kernels.
inline bool fused_shape_ok(const void* W, int rows, int cols, int ldw, int block) {
  return cols % 8 == 0 && ldw % 8 == 0 && aligned_to(W, 16) && cols <= kFusedMaxCols && rows / block <= kFusedMaxBlocks;
}

#ifdef __CUDACC__
__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) {
  return __uint_as_float(static_cast<uint32_t>(b) << 16);
}

// Sum of squares of one group in float32, elements taken in increasing index order starting
// from +0.  The square of a bf16 value is exact in float32, so the fused multiply-add rounds
// exactly once per element, the same as a separate multiply and add would.
__device__ __forceinline__ float group_sumsq_strided(const uint16_t* __restrict__ p, int n, size_t stride) {
  float acc = 0.0f;
  for (int e = 0; e < n; ++e) {
    const float w = bf16_bits_to_float(p[static_cast<size_t>(e) * stride]);
    acc = __fmaf_rn(w, w, acc);
  }
  return acc;
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Float32 sums of squares of 8 adjacent columns over the d rows of a row-block: eight independent
// sequential chains, each the defined decision quantity of its group.
template <int ROWS>
__device__ __forceinline__ void sumsq8_rows(const uint16_t* __restrict__ p, int ldw, float (&acc)[8]) {
  uint4 v[ROWS];
#pragma unroll
  for (int u = 0; u < ROWS; ++u) v[u] = __ldg(reinterpret_cast<const uint4*>(p + static_cast<size_t>(u) * ldw));
#pragma unroll
  for (int u = 0; u < ROWS; ++u) {     // rows in increasing order: the chains stay sequential
    const uint32_t w32[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float lo = __uint_as_float(w32[i] << 16), hi = __uint_as_float(w32[i] & 0xffff0000u);
      acc[2 * i] = __fmaf_rn(lo, lo, acc[2 * i]);
      acc[2 * i + 1] = __fmaf_rn(hi, hi, acc[2 * i + 1]);
    }
  }
}
__device__ __forceinline__ void sumsq8(const uint16_t* __restrict__ p, int d, int ldw, float (&acc)[8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0.0f;
  int r = 0;
  for (; r + 16 <= d; r += 16) sumsq8_rows<16>(p + static_cast<size_t>(r) * ldw, ldw, acc);   // 256 bytes in flight
  for (; r + 4 <= d; r += 4) sumsq8_rows<4>(p + static_cast<size_t>(r) * ldw, ldw, acc);
  for (; r < d; ++r) sumsq8_rows<1>(p + static_cast<size_t>(r) * ldw, ldw, acc);
}

// Block-wide exclusive prefix sum of one int per thread (blockDim.x a multiple of 32, <= 1024).
__device__ __forceinline__ int block_exclusive_scan(int v, int* s_warp, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int up = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += up;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = lane < n_warps ? s_warp[lane] : 0;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, w, o);
      if (lane >= o) w += up;
    }
    s_warp[lane] = w;  // inclusive totals of warps
  }
  __syncthreads();
  const int before = warp ? s_warp[warp - 1] : 0;
  *total = s_warp[n_warps - 1];
  __syncthreads();  // s_warp may be reused by the caller's next round
  return before + incl - v;
}

// Norm and reciprocal of the reported (not the deciding) quantities: the hardware's approximate square
// root and reciprocal, each within about one unit in the last place of float32, far inside the 1e-5
// these outputs are held to, at a sixth of the instructions of the correctly rounded forms.  Every
// kernel that writes norms or gamma goes through these two, so all of them give the same bits.
__device__ __forceinline__ float norm_from_sumsq(float S) {
  float n;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(n) : "f"(S));
  return n;
}
__device__ __forceinline__ float reciprocal(float x) {
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}

struct NormOut {
  float* norms;
  const float* gamma_in;
  float* gamma_out;
  double* penalty;
  float eps;
  int squared;  // 0: gamma = 1/(n+eps), term gamma*n ; 1: alpha = 1/(S+eps), term alpha*S
};

// Finishes one group from its float32 sum of squares; returns the group's penalty term.
__device__ __forceinline__ double finish_group(const NormOut& o, size_t g, float S) {
  const float n = norm_from_sumsq(S);
  const float base = o.squared ? S : n;
  const float fresh = reciprocal(base + o.eps);
  if (o.norms) o.norms[g] = n;
  if (o.gamma_out) o.gamma_out[g] = fresh;
  const float weight = o.gamma_in ? o.gamma_in[g] : fresh;
  return static_cast<double>(weight) * static_cast<double>(base);
}

#endif  // __CUDACC__

}  // namespace bsp
