// bsp_group_norms: per-group l2 norms, the gamma update and the reweighted group-Lasso penalty
// (Section 3.2, Eq. 2 and Eq. 3) in a single pass over W.  Bandwidth-bound: every weight is
// read once, one float is written per group and per requested output.
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

// Orientation C fast path: one thread owns 8 adjacent columns of one row-block and walks its d
// rows with 16-byte loads (a warp covers 512 contiguous bytes of every row).  The eight sums
// are independent sequential chains, so each equals the defined float32 decision quantity.
template <int UNROLL>
__global__ void __launch_bounds__(256)
norms_c_vec8_kernel(const uint16_t* __restrict__ W, int n_blocks, int cols, int ldw, int d, NormOut o) {
  const int chunks = cols >> 3;
  const long long item = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  double local = 0.0;
  if (item < static_cast<long long>(n_blocks) * chunks) {
    const int b = static_cast<int>(item / chunks);
    const int q = static_cast<int>(item - static_cast<long long>(b) * chunks);
    const uint16_t* p = W + static_cast<size_t>(b) * d * ldw + (q << 3);
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.0f;
    int r = 0;
    for (; r + UNROLL <= d; r += UNROLL) {
      uint4 v[UNROLL];
#pragma unroll
      for (int u = 0; u < UNROLL; ++u)
        v[u] = __ldg(reinterpret_cast<const uint4*>(p + static_cast<size_t>(r + u) * ldw));
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        const uint32_t w32[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float lo = __uint_as_float(w32[i] << 16);
          const float hi = __uint_as_float(w32[i] & 0xffff0000u);
          acc[2 * i] = __fmaf_rn(lo, lo, acc[2 * i]);
          acc[2 * i + 1] = __fmaf_rn(hi, hi, acc[2 * i + 1]);
        }
      }
    }
    for (; r < d; ++r) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(p + static_cast<size_t>(r) * ldw));
      const uint32_t w32[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float lo = __uint_as_float(w32[i] << 16);
        const float hi = __uint_as_float(w32[i] & 0xffff0000u);
        acc[2 * i] = __fmaf_rn(lo, lo, acc[2 * i]);
        acc[2 * i + 1] = __fmaf_rn(hi, hi, acc[2 * i + 1]);
      }
    }
    const size_t g0 = static_cast<size_t>(b) * cols + (q << 3);
#pragma unroll
    for (int i = 0; i < 8; ++i) local += finish_group(o, g0 + i, acc[i]);
  }
  add_penalty(o, local);
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
  const bool vec_ok = orient == BSP_ORIENT_C && (cols % 8 == 0) && (ldw % 8 == 0) && aligned_to(W, 16);
  if (vec_ok) {
    const long long items = static_cast<long long>(rows / block) * (cols / 8);
    const unsigned grid = static_cast<unsigned>((items + 255) / 256);
    if (block % 8 == 0)
      norms_c_vec8_kernel<8><<<grid, 256, 0, s>>>(w, rows / block, cols, ldw, block, o);
    else
      norms_c_vec8_kernel<4><<<grid, 256, 0, s>>>(w, rows / block, cols, ldw, block, o);
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
