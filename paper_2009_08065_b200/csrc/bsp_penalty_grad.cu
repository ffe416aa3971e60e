// bsp_penalty_grad: gradient of the reweighted group-Lasso term with respect to W, the penalty
// weights held fixed (Algorithm 2 keeps gamma between milestones while the optimiser minimises
// mixed_loss = l1loss + f(W, b)):
//   Eq. 2 / Eq. 3 form:   d/dW_e [ gamma_g ||W_g||_2 ] = gamma_g W_e / ||W_g||_2   (0 for an all-zero group)
//   squared-norm variant: d/dW_e [ alpha_g ||W_g||^2 ] = 2 alpha_g W_e
// HBM-bound: W is read (the second read of a group hits L1/L2), one float is written per weight.
#include "bsp_common.cuh"

namespace bsp {
namespace {

struct GradArgs {
  const uint16_t* W;
  int rows, cols, ldw, block, orient, squared, accumulate;
  const float* gamma;
  float scale;
  float* grad;
  int ldg;
};

// Orientation C, 8-element alignment: one thread per 8 adjacent columns of a row-block.
__global__ void __launch_bounds__(256)
grad_c_vec8_kernel(GradArgs A) {
  const int chunks = A.cols >> 3;
  const long long item = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (item >= static_cast<long long>(A.rows / A.block) * chunks) return;
  const int b = static_cast<int>(item / chunks), q = static_cast<int>(item - static_cast<long long>(b) * chunks);
  const uint16_t* p = A.W + static_cast<size_t>(b) * A.block * A.ldw + (q << 3);
  float factor[8];
  const float4 g0 = __ldg(reinterpret_cast<const float4*>(A.gamma + static_cast<size_t>(b) * A.cols + (q << 3)));
  const float4 g1 = __ldg(reinterpret_cast<const float4*>(A.gamma + static_cast<size_t>(b) * A.cols + (q << 3) + 4));
  const float gam[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
  if (A.squared) {
#pragma unroll
    for (int i = 0; i < 8; ++i) factor[i] = 2.0f * A.scale * gam[i];
  } else {
    float acc[8];
    sumsq8(p, A.block, A.ldw, acc);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float n = __fsqrt_rn(acc[i]);
      factor[i] = n > 0.0f ? __fdiv_rn(A.scale * gam[i], n) : 0.0f;
    }
  }
  for (int r = 0; r < A.block; ++r) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(p + static_cast<size_t>(r) * A.ldw));
    const uint32_t w32[4] = {v.x, v.y, v.z, v.w};
    float o[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      o[2 * i] = factor[2 * i] * __uint_as_float(w32[i] << 16);
      o[2 * i + 1] = factor[2 * i + 1] * __uint_as_float(w32[i] & 0xffff0000u);
    }
    float4* dst = reinterpret_cast<float4*>(A.grad + (static_cast<size_t>(b) * A.block + r) * A.ldg + (q << 3));
    if (A.accumulate) {
      const float4 a = dst[0], c = dst[1];
      o[0] += a.x; o[1] += a.y; o[2] += a.z; o[3] += a.w;
      o[4] += c.x; o[5] += c.y; o[6] += c.z; o[7] += c.w;
    }
    dst[0] = make_float4(o[0], o[1], o[2], o[3]);
    dst[1] = make_float4(o[4], o[5], o[6], o[7]);
  }
}

// Any geometry: one thread per group.
__global__ void __launch_bounds__(256)
grad_generic_kernel(GradArgs A) {
  const bool c_orient = A.orient == BSP_ORIENT_C;
  const long long n_groups = c_orient ? static_cast<long long>(A.rows / A.block) * A.cols
                                      : static_cast<long long>(A.rows) * (A.cols / A.block);
  const long long g = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (g >= n_groups) return;
  size_t first, stride;
  if (c_orient) {
    const long long b = g / A.cols;
    first = static_cast<size_t>(b) * A.block * A.ldw + static_cast<size_t>(g - b * A.cols);
    stride = A.ldw;
  } else {
    const int per_row = A.cols / A.block;
    const long long i = g / per_row;
    first = static_cast<size_t>(i) * A.ldw + static_cast<size_t>(g - i * per_row) * A.block;
    stride = 1;
  }
  float factor;
  if (A.squared) {
    factor = 2.0f * A.scale * A.gamma[g];
  } else {
    const float n = __fsqrt_rn(group_sumsq_strided(A.W + first, A.block, stride));
    factor = n > 0.0f ? __fdiv_rn(A.scale * A.gamma[g], n) : 0.0f;
  }
  // the same element position in grad: row = first / ldw, col = first % ldw
  const size_t row0 = first / A.ldw, col0 = first - row0 * A.ldw;
  for (int e = 0; e < A.block; ++e) {
    const size_t row = c_orient ? row0 + e : row0, col = c_orient ? col0 : col0 + e;
    const float v = factor * bf16_bits_to_float(A.W[first + e * stride]);
    float* dst = A.grad + row * A.ldg + col;
    *dst = A.accumulate ? *dst + v : v;
  }
}

}  // namespace
}  // namespace bsp

extern "C" int bsp_penalty_grad(const void* W, int rows, int cols, int ldw, int block, int orient, int pen,
                                const float* gamma, float scale, float* grad, int ldg, int accumulate,
                                void* stream) {
  using namespace bsp;
  int st = check_matrix_args(W, rows, cols, ldw, block, orient);
  if (st != BSP_OK) return st;
  if (pen != BSP_PEN_L2 && pen != BSP_PEN_L2SQ) return BSP_ERR_ARG;
  if (gamma == nullptr || grad == nullptr || !aligned_to(grad, 4) || !aligned_to(gamma, 4)) return BSP_ERR_ARG;
  if (scale != scale) return BSP_ERR_ARG;
  if (ldg < cols) return BSP_ERR_SHAPE;
  GradArgs A{static_cast<const uint16_t*>(W), rows, cols, ldw, block, orient, pen == BSP_PEN_L2SQ ? 1 : 0,
             accumulate ? 1 : 0, gamma, scale, grad, ldg};
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const bool vec = orient == BSP_ORIENT_C && cols % 8 == 0 && ldw % 8 == 0 && ldg % 4 == 0 && aligned_to(W, 16) &&
                   aligned_to(grad, 16) && aligned_to(gamma, 16);
  if (vec) {
    const long long items = static_cast<long long>(rows / block) * (cols / 8);
    grad_c_vec8_kernel<<<static_cast<unsigned>((items + 255) / 256), 256, 0, s>>>(A);
  } else {
    int nb, ng;
    geometry(rows, cols, block, orient, &nb, &ng);
    const long long groups = static_cast<long long>(nb) * ng;
    grad_generic_kernel<<<static_cast<unsigned>((groups + 255) / 256), 256, 0, s>>>(A);
  }
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}
