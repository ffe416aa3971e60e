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
#endif  // __CUDACC__

}  // namespace bsp
