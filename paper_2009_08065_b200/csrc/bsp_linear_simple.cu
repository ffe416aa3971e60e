// bsp_linear_cuda_core: the pruned linear layer evaluated directly from the canonical packed
// form on CUDA cores, one thread per output.  Row-block b reads only the X columns listed in
// its index list.  This is the path for shapes the tensor-core kernel does not accept and the
// in-library cross-check for it; it is not tuned.
#include <math.h>

#include "bsp_common.cuh"

namespace bsp {
namespace {

__global__ void __launch_bounds__(256)
linear_simple_kernel(const int32_t* __restrict__ blk_ptr, const int32_t* __restrict__ idx,
                     const uint16_t* __restrict__ vals, int n_out, int block,
                     const uint16_t* __restrict__ X, int tokens, int ldx,
                     const uint16_t* __restrict__ bias, int act, uint16_t* __restrict__ Y, int ldy) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  const int t = blockIdx.y;
  if (n >= n_out || t >= tokens) return;
  const int b = n / block, r = n - b * block;
  const int lo = blk_ptr[b], kc = blk_ptr[b + 1] - lo;
  const uint16_t* wrow = vals + static_cast<size_t>(block) * lo + static_cast<size_t>(r) * kc;
  const int32_t* cols = idx + lo;
  const uint16_t* xrow = X + static_cast<size_t>(t) * ldx;
  float acc = 0.0f;
  for (int j = 0; j < kc; ++j)
    acc = __fmaf_rn(bf16_bits_to_float(xrow[cols[j]]), bf16_bits_to_float(wrow[j]), acc);
  if (bias) acc += bf16_bits_to_float(bias[n]);
  if (act == BSP_ACT_GELU) acc = 0.5f * acc * (1.0f + erff(acc * 0.70710678118654752440f));
  Y[static_cast<size_t>(t) * ldy + n] = __bfloat16_as_ushort(__float2bfloat16_rn(acc));
}

}  // namespace

int check_linear_args(const void* a, const void* b, const void* c, int n_out, int k_in, int block,
                      const void* X, int tokens, int ldx, int act, const void* Y, int ldy) {
  if (a == nullptr || b == nullptr || c == nullptr || X == nullptr || Y == nullptr) return BSP_ERR_ARG;
  if (n_out <= 0 || k_in <= 0 || block <= 0 || tokens < 0) return BSP_ERR_ARG;
  if (act != BSP_ACT_NONE && act != BSP_ACT_GELU) return BSP_ERR_ARG;
  if (n_out % block) return BSP_ERR_SHAPE;
  if (ldx < k_in || ldy < n_out) return BSP_ERR_SHAPE;
  return BSP_OK;
}

}  // namespace bsp

extern "C" int bsp_linear_cuda_core(const int32_t* blk_ptr, const int32_t* idx, const void* vals,
                                    int n_out, int k_in, int block, const void* X, int tokens, int ldx,
                                    const void* bias, int act, void* Y, int ldy, void* stream) {
  using namespace bsp;
  int st = check_linear_args(blk_ptr, idx, vals, n_out, k_in, block, X, tokens, ldx, act, Y, ldy);
  if (st != BSP_OK) return st;
  if (tokens == 0) return BSP_OK;
  if (tokens > 65535 * 1) {
    // grid.y limit: split the token range
    for (int t0 = 0; t0 < tokens; t0 += 65535) {
      const int nt = tokens - t0 < 65535 ? tokens - t0 : 65535;
      st = bsp_linear_cuda_core(blk_ptr, idx, vals, n_out, k_in, block,
                                static_cast<const uint16_t*>(X) + static_cast<size_t>(t0) * ldx, nt, ldx, bias, act,
                                static_cast<uint16_t*>(Y) + static_cast<size_t>(t0) * ldy, ldy, stream);
      if (st != BSP_OK) return st;
    }
    return BSP_OK;
  }
  dim3 grid((n_out + 255) / 256, tokens);
  linear_simple_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      blk_ptr, idx, static_cast<const uint16_t*>(vals), n_out, block, static_cast<const uint16_t*>(X), tokens,
      ldx, static_cast<const uint16_t*>(bias), act, static_cast<uint16_t*>(Y), ldy);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}
