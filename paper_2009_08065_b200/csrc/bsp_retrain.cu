// Algorithm 2's retraining loop on the device: "update W ... using Adam", then "W = W * Mask", in
// one pass (bsp_masked_adam_step), and the refresh of the packed values of Section 3.1's storage
// under the fixed kept sets (bsp_repack_values); and the mask loop itself (bsp_dense_mask).
//
// Adam is taken as published (Kingma & Ba 2015, with bias correction); the paper gives no
// hyper-parameters beyond the learning rate, so they are the caller's.  The weights that the
// optimiser owns are float32 (a bf16 weight of size 0.02 cannot absorb a step of 3e-5); the bf16
// copy that the linear layer reads, already multiplied by the mask, is written in the same pass:
// it IS the zero-expanded execution layout of bsp_linear_planned.
// HBM-bound, one thread per 4 adjacent weights: 16 bytes of gradient, weight and both moments in,
// weight and moments out plus the bf16 copy: 16 + 12 + 2 = 30 bytes per weight.
#include <math.h>

#include "bsp_common.cuh"

namespace bsp {
namespace {

struct AdamArgs {
  float* W;
  const float* G;
  float* M;
  float* V;
  int rows, cols, ldw, ldg;
  const uint8_t* keep;       // per-group flags, or null (no mask)
  int block, orient;
  float lr, beta1, beta2, eps, decay;
  float inv_c1, inv_c2;      // 1 / (1 - beta^step)
  uint16_t* Wb;              // bf16 copy, or null
  int ldb;
};

__global__ void __launch_bounds__(256)
masked_adam_kernel(AdamArgs A) {
  const int quads = A.cols >> 2;
  const long long item = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (item >= static_cast<long long>(A.rows) * quads) return;
  const int r = static_cast<int>(item / quads), c = static_cast<int>(item - static_cast<long long>(r) * quads) << 2;
  const size_t iw = static_cast<size_t>(r) * A.ldw + c, ig = static_cast<size_t>(r) * A.ldg + c;
  const float4 w4 = *reinterpret_cast<const float4*>(A.W + iw);
  const float4 g4 = __ldg(reinterpret_cast<const float4*>(A.G + ig));
  const float4 m4 = *reinterpret_cast<const float4*>(A.M + iw);
  const float4 v4 = *reinterpret_cast<const float4*>(A.V + iw);
  float w[4] = {w4.x, w4.y, w4.z, w4.w};
  const float g[4] = {g4.x, g4.y, g4.z, g4.w};
  float m[4] = {m4.x, m4.y, m4.z, m4.w};
  float v[4] = {v4.x, v4.y, v4.z, v4.w};
  uint32_t keep[4] = {1u, 1u, 1u, 1u};
  if (A.keep != nullptr) {
    if (A.orient == BSP_ORIENT_C) {
      const uint8_t* f = A.keep + static_cast<size_t>(r / A.block) * A.cols + c;
#pragma unroll
      for (int i = 0; i < 4; ++i) keep[i] = f[i];
    } else {
      const uint8_t* f = A.keep + static_cast<size_t>(r) * (A.cols / A.block);
#pragma unroll
      for (int i = 0; i < 4; ++i) keep[i] = f[(c + i) / A.block];
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    m[i] = __fmaf_rn(A.beta1, m[i], (1.0f - A.beta1) * g[i]);
    v[i] = __fmaf_rn(A.beta2, v[i], (1.0f - A.beta2) * g[i] * g[i]);
    const float mhat = m[i] * A.inv_c1, vhat = v[i] * A.inv_c2;
    const float upd = __fdiv_rn(mhat, __fsqrt_rn(vhat) + A.eps) + A.decay * w[i];
    w[i] = keep[i] ? __fmaf_rn(-A.lr, upd, w[i]) : 0.0f;
  }
  *reinterpret_cast<float4*>(A.W + iw) = make_float4(w[0], w[1], w[2], w[3]);
  *reinterpret_cast<float4*>(A.M + iw) = make_float4(m[0], m[1], m[2], m[3]);
  *reinterpret_cast<float4*>(A.V + iw) = make_float4(v[0], v[1], v[2], v[3]);
  if (A.Wb != nullptr) {
    uint32_t lo, hi;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(lo) : "f"(w[1]), "f"(w[0]));
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(hi) : "f"(w[3]), "f"(w[2]));
    *reinterpret_cast<uint2*>(A.Wb + static_cast<size_t>(r) * A.ldb + c) = make_uint2(lo, hi);
  }
}

// One CTA per row-block: tile[r][p] = W[b*d + r][idx[lo + p]]; the stores are contiguous.
__global__ void __launch_bounds__(256)
repack_kernel(const uint16_t* __restrict__ W, int ldw, int block, const int32_t* __restrict__ blk_ptr,
              const int32_t* __restrict__ idx, uint16_t* __restrict__ vals) {
  const int b = blockIdx.x;
  const int lo = blk_ptr[b], kc = blk_ptr[b + 1] - lo;
  const uint16_t* wblk = W + static_cast<size_t>(b) * block * ldw;
  uint16_t* tile = vals + static_cast<size_t>(block) * lo;
  const int r_lo = blockIdx.y * 4, r_hi = min(block, r_lo + 4);
  for (int r = r_lo; r < r_hi; ++r)
    for (int p = threadIdx.x; p < kc; p += blockDim.x)
      tile[static_cast<size_t>(r) * kc + p] = wblk[static_cast<size_t>(r) * ldw + __ldg(idx + lo + p)];
}

// Algorithm 2's mask loop: Mask_ij = 0 if W_ij == 0 else 1 (either sign of zero is zero).
__global__ void __launch_bounds__(256)
dense_mask_kernel(const uint16_t* __restrict__ W, int rows, int cols, int ldw, uint8_t* __restrict__ mask, int ldm) {
  const long long e = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (e >= static_cast<long long>(rows) * cols) return;
  const int r = static_cast<int>(e / cols), c = static_cast<int>(e - static_cast<long long>(r) * cols);
  mask[static_cast<size_t>(r) * ldm + c] = (W[static_cast<size_t>(r) * ldw + c] & 0x7fffu) != 0 ? 1 : 0;
}

}  // namespace
}  // namespace bsp

extern "C" int bsp_dense_mask(const void* W, int rows, int cols, int ldw, uint8_t* mask, int ldm, void* stream) {
  using namespace bsp;
  if (W == nullptr || mask == nullptr || rows <= 0 || cols <= 0) return BSP_ERR_ARG;
  if (ldw < cols || ldm < cols) return BSP_ERR_SHAPE;
  const long long elems = static_cast<long long>(rows) * cols;
  const long long blocks = (elems + 255) / 256;
  if (blocks > 0x7fffffffLL) return BSP_ERR_UNSUPPORTED;
  dense_mask_kernel<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint16_t*>(W), rows, cols, ldw, mask, ldm);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

extern "C" int bsp_masked_adam_step(float* W, const float* grad, float* m, float* v, int rows, int cols, int ldw,
                                    int ldg, const uint8_t* keep, int block, int orient, float lr, float beta1,
                                    float beta2, float eps, float weight_decay, int step, void* W_bf16, int ldb,
                                    void* stream) {
  using namespace bsp;
  if (W == nullptr || grad == nullptr || m == nullptr || v == nullptr) return BSP_ERR_ARG;
  if (rows <= 0 || cols <= 0 || step < 1) return BSP_ERR_ARG;
  if (!(beta1 >= 0.0f && beta1 < 1.0f) || !(beta2 >= 0.0f && beta2 < 1.0f) || !(eps >= 0.0f) || !(lr == lr) ||
      !(weight_decay == weight_decay))
    return BSP_ERR_ARG;
  if (ldw < cols || ldg < cols || (W_bf16 != nullptr && ldb < cols)) return BSP_ERR_SHAPE;
  if (keep != nullptr) {
    if (block <= 0 || (orient != BSP_ORIENT_C && orient != BSP_ORIENT_R)) return BSP_ERR_ARG;
    int nb, ng;
    if (!geometry(rows, cols, block, orient, &nb, &ng)) return BSP_ERR_SHAPE;
  }
  if (cols % 4 || ldw % 4 || ldg % 4 || !aligned_to(W, 16) || !aligned_to(grad, 16) || !aligned_to(m, 16) ||
      !aligned_to(v, 16) || (W_bf16 != nullptr && (ldb % 4 || !aligned_to(W_bf16, 8))))
    return BSP_ERR_UNSUPPORTED;
  AdamArgs A;
  A.W = W; A.G = grad; A.M = m; A.V = v;
  A.rows = rows; A.cols = cols; A.ldw = ldw; A.ldg = ldg;
  A.keep = keep; A.block = block; A.orient = orient;
  A.lr = lr; A.beta1 = beta1; A.beta2 = beta2; A.eps = eps; A.decay = weight_decay;
  // bias corrections in double on the host, rounded once
  A.inv_c1 = static_cast<float>(1.0 / (1.0 - pow(static_cast<double>(beta1), step)));
  A.inv_c2 = static_cast<float>(1.0 / (1.0 - pow(static_cast<double>(beta2), step)));
  A.Wb = static_cast<uint16_t*>(W_bf16);
  A.ldb = ldb;
  const long long items = static_cast<long long>(rows) * (cols >> 2);
  const long long blocks = (items + 255) / 256;
  if (blocks > 0x7fffffffLL) return BSP_ERR_UNSUPPORTED;
  masked_adam_kernel<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(A);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

extern "C" int bsp_repack_values(const void* W, int rows, int cols, int ldw, int block, const int32_t* blk_ptr,
                                 const int32_t* idx, void* vals, void* stream) {
  using namespace bsp;
  if (blk_ptr == nullptr || idx == nullptr || vals == nullptr) return BSP_ERR_ARG;
  int st = check_matrix_args(W, rows, cols, ldw, block, BSP_ORIENT_C);
  if (st != BSP_OK) return st;
  const int nb = rows / block;
  const dim3 grid(nb, (block + 3) / 4);
  if (grid.y > 65535) return BSP_ERR_UNSUPPORTED;
  repack_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const uint16_t*>(W), ldw, block, blk_ptr,
                                                                    idx, static_cast<uint16_t*>(vals));
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}
