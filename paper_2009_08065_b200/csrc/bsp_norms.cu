// bsp_group_norms: per-group l2 norms, the gamma update and the reweighted group-Lasso penalty
// (Section 3.2, Eq. 2 and Eq. 3) in a single pass over W.  Bandwidth-bound: every weight is
// read once, one float is written per group and per requested output.  Orientation C with
// 8-element alignment runs the vectorised stage-1 kernel of bsp_fused.cu; this file holds the
// generic kernel (any alignment, orientation R) and the entry point.
#include "bsp_common.cuh"

namespace bsp {

int& last_cuda_error_ref() {
  static thread_local int e = 0;
  return e;
}

namespace {

__device__ __forceinline__ void add_penalty(const NormOut& o, double local) {
  if (o.penalty == nullptr) return;  // uniform across the grid
  local = warp_sum(local);
  if ((threadIdx.x & 31) == 0 && local != 0.0) atomicAdd(o.penalty, local);
}

// Any geometry: one thread per group.  C: lanes run along columns (each row is read
// contiguously by the warp).  R: lanes run along the strips of one row (adjacent groups are
// adjacent in memory).
__global__ void __launch_bounds__(256)
norms_generic_kernel(const uint16_t* __restrict__ W, int rows, int cols, int ldw, int block, int orient,
                     NormOut o) {
  const long long n_groups = (orient == BSP_ORIENT_C) ? static_cast<long long>(rows / block) * cols
                                                      : static_cast<long long>(rows) * (cols / block);
  const long long g = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  double local = 0.0;
  if (g < n_groups) {
    float S;
    if (orient == BSP_ORIENT_C) {
      const long long b = g / cols;
      const int j = static_cast<int>(g - b * cols);
      S = group_sumsq_strided(W + static_cast<size_t>(b) * block * ldw + j, block, ldw);
    } else {
      const int per_row = cols / block;
      const long long i = g / per_row;
      const int a = static_cast<int>(g - i * per_row);
      S = group_sumsq_strided(W + static_cast<size_t>(i) * ldw + static_cast<size_t>(a) * block, block, 1);
    }
    local = finish_group(o, static_cast<size_t>(g), S);
  }
  add_penalty(o, local);
}

}  // namespace
}  // namespace bsp

extern "C" const char* bsp_status_string(int status) {
  switch (status) {
    case BSP_OK: return "BSP_OK";
    case BSP_ERR_ARG: return "BSP_ERR_ARG: invalid argument";
    case BSP_ERR_SHAPE: return "BSP_ERR_SHAPE: block does not divide the matrix, or a leading dimension is too small";
    case BSP_ERR_WORKSPACE: return "BSP_ERR_WORKSPACE: workspace too small";
    case BSP_ERR_CUDA: return "BSP_ERR_CUDA: a CUDA call failed";
    case BSP_ERR_TIMEOUT: return "BSP_ERR_TIMEOUT: a bounded device-side wait expired";
    case BSP_ERR_UNSUPPORTED: return "BSP_ERR_UNSUPPORTED: size beyond a documented limit";
    default: return "unknown bsp status";
  }
}

extern "C" int bsp_last_cuda_error(void) { return bsp::last_cuda_error_ref(); }

extern "C" int bsp_group_norms(const void* W, int rows, int cols, int ldw, int block, int orient,
                               float eps, int pen, float* norms, const float* gamma_in,
                               float* gamma_out, double* penalty, void* stream) {
  using namespace bsp;
  int st = check_matrix_args(W, rows, cols, ldw, block, orient);
  if (st != BSP_OK) return st;
  if (pen != BSP_PEN_L2 && pen != BSP_PEN_L2SQ) return BSP_ERR_ARG;
  if (!(eps >= 0.0f)) return BSP_ERR_ARG;
  if (norms == nullptr && gamma_out == nullptr && penalty == nullptr) return BSP_ERR_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (penalty) BSP_CUDA_TRY(cudaMemsetAsync(penalty, 0, sizeof(double), s));

  NormOut o{norms, gamma_in, gamma_out, penalty, eps, pen == BSP_PEN_L2SQ ? 1 : 0};
  const uint16_t* w = static_cast<const uint16_t*>(W);
  const bool vec_ok = orient == BSP_ORIENT_C && cols % 8 == 0 && ldw % 8 == 0 && aligned_to(W, 16) &&   // stage 1 alone has no size limit
                      (norms == nullptr || aligned_to(norms, 16)) && (gamma_out == nullptr || aligned_to(gamma_out, 16)) &&
                      (gamma_in == nullptr || aligned_to(gamma_in, 16));
  if (vec_ok) {
    // vectorised stage 1 with the keep decision switched off; the penalty is added by atomics
    FusedJob j{w, rows, cols, ldw, rows / block, 0.0f, nullptr, norms, gamma_in, gamma_out, penalty,
               nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    return fused_stage1(&j, 1, block, eps, o.squared, s);
  } else {
    int nb, ng;
    geometry(rows, cols, block, orient, &nb, &ng);
    const long long groups = static_cast<long long>(nb) * ng;
    const unsigned grid = static_cast<unsigned>((groups + 255) / 256);
    norms_generic_kernel<<<grid, 256, 0, s>>>(w, rows, cols, ldw, block, orient, o);
  }
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}
