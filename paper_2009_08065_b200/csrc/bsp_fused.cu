// bsp_prepare_batched: for a batch of weight matrices (orientation C), everything the path does
// on the weight side in two launches — (1) group norms, gamma, penalty partials, keep flags and
// per-block counts in one pass over W; (2) blk_ptr, ascending index lists, packed tiles, the
// penalty total, and (optionally) the linear layer's execution layout.  Results are bit-identical
// to bsp_group_norms + bsp_prune_pack + bsp_linear_plan called per matrix (the penalty up to its
// summation order, which here is fixed, so it is reproducible run to run).
#include "bsp_common.cuh"

namespace bsp {
namespace {

constexpr int kMaxJobs = 16;
constexpr int kThreads = 256;

struct Job {
  const uint16_t* W;
  int rows, cols, ldw, n_blocks;
  float threshold;
  const float* threshold_dev;
  NormOut out;                 // norms / gamma_in / gamma_out / (penalty unused here) / eps / squared
  double* penalty;
  uint8_t* flags;
  int32_t* counts;
  double* partial;             // per-block penalty partial sums
  int32_t* blk_ptr;
  int32_t* idx;
  uint16_t* vals;
  int64_t* kept_weights;
  uint16_t* plan;
};

struct Batch {
  int n_jobs, block;
  int first_block[kMaxJobs + 1];   // CTA index of each job's first row-block
  Job job[kMaxJobs];
};

__device__ __forceinline__ int find_job(const Batch& B, int cta) {
  int j = 0;
  while (j + 1 < B.n_jobs && cta >= B.first_block[j + 1]) ++j;
  return j;
}

// (1) one CTA per row-block of some job; one thread per 8 adjacent columns.
__global__ void __launch_bounds__(kThreads)
fused_norms_flags_kernel(const __grid_constant__ Batch B) {
  __shared__ int s_cnt[kThreads / 32];
  __shared__ double s_pen[kThreads / 32];
  const int j = find_job(B, blockIdx.x);
  const Job& J = B.job[j];
  const int b = blockIdx.x - B.first_block[j];
  const float t = J.threshold_dev ? *J.threshold_dev : J.threshold;
  const bool keep_all = t < 0.0f;
  const float t2 = __fmul_rn(t, t);
  const bool want_norms = J.out.norms || J.out.gamma_out || J.penalty;
  NormOut o = J.out;
  int count = 0;
  double pen = 0.0;
  for (int q = threadIdx.x; q < (J.cols >> 3); q += blockDim.x) {
    float acc[8];
    sumsq8(J.W + static_cast<size_t>(b) * B.block * J.ldw + (q << 3), B.block, J.ldw, acc);
    uint32_t lo = 0, hi = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t k0 = (keep_all || acc[i] > t2) ? 1u : 0u;
      const uint32_t k1 = (keep_all || acc[4 + i] > t2) ? 1u : 0u;
      lo |= k0 << (8 * i);
      hi |= k1 << (8 * i);
      count += static_cast<int>(k0 + k1);
    }
    const size_t g0 = static_cast<size_t>(b) * J.cols + (q << 3);
    *reinterpret_cast<uint2*>(J.flags + g0) = make_uint2(lo, hi);
    if (want_norms) {
#pragma unroll
      for (int i = 0; i < 8; ++i) pen += finish_group(o, g0 + i, acc[i]);
    }
  }
  count = warp_sum(count);
  pen = warp_sum(pen);
  const int warp = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) { s_cnt[warp] = count; s_pen[warp] = pen; }
  __syncthreads();
  if (threadIdx.x == 0) {
    int c = 0;
    double p = 0.0;
    for (int w = 0; w < kThreads / 32; ++w) { c += s_cnt[w]; p += s_pen[w]; }   // fixed order
    J.counts[b] = c;
    J.partial[b] = p;
  }
}

// (2) grid = (row-blocks of all jobs, row splits).
__global__ void __launch_bounds__(kThreads)
fused_compact_plan_kernel(const __grid_constant__ Batch B) {
  extern __shared__ int32_t s_idx[];   // kept column indices of this block, ascending
  __shared__ int s_warp[32];
  __shared__ double s_red[kThreads / 32];
  __shared__ int s_base;
  const int j = find_job(B, blockIdx.x);
  const Job& J = B.job[j];
  const int b = blockIdx.x - B.first_block[j];
  const int d = B.block;

  // penalty total of the job: block 0 / split 0 adds the per-block partials in a fixed order
  if (b == 0 && blockIdx.y == 0 && J.penalty != nullptr) {
    double p = 0.0;
    for (int i = threadIdx.x; i < J.n_blocks; i += blockDim.x) p += J.partial[i];
    p = warp_sum(p);
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = p;
    __syncthreads();
    if (threadIdx.x == 0) {
      double tot = 0.0;
      for (int w = 0; w < kThreads / 32; ++w) tot += s_red[w];
      *J.penalty = tot;
    }
  }

  // blk_ptr[b] = sum of counts[0..b)
  int part = 0;
  for (int i = threadIdx.x; i < b; i += blockDim.x) part += J.counts[i];
  part = warp_sum(part);
  if (threadIdx.x == 0) s_base = 0;
  __syncthreads();
  if ((threadIdx.x & 31) == 0 && part) atomicAdd(&s_base, part);
  __syncthreads();
  const int base = s_base;
  const int kc = J.counts[b];
  if (blockIdx.y == 0 && threadIdx.x == 0) {
    J.blk_ptr[b] = base;
    if (b == J.n_blocks - 1) {
      J.blk_ptr[J.n_blocks] = base + kc;
      if (J.kept_weights) *J.kept_weights = static_cast<int64_t>(base + kc) * d;
    }
  }

  const int rows_per = (d + gridDim.y - 1) / gridDim.y;
  const int r_lo = blockIdx.y * rows_per;
  const int r_hi = min(d, r_lo + rows_per);
  const uint16_t* wblk = J.W + static_cast<size_t>(b) * d * J.ldw;
  const uint8_t* flags = J.flags + static_cast<size_t>(b) * J.cols;
  const int chunks = J.cols >> 3;

  // execution layout: W with the pruned columns of this row-block zeroed, 16 bytes at a time
  if (J.plan != nullptr) {
    for (int e = threadIdx.x; e < (r_hi - r_lo) * chunks; e += blockDim.x) {
      const int r = r_lo + e / chunks, q = e % chunks;
      const uint2 f = *reinterpret_cast<const uint2*>(flags + (q << 3));
      uint4 w = __ldg(reinterpret_cast<const uint4*>(wblk + static_cast<size_t>(r) * J.ldw + (q << 3)));
      // a flag byte is 0 or 1: (flag * 0xffff) masks the matching 16-bit element
      w.x &= ((f.x & 0xffu) * 0xffffu) | (((f.x >> 8) & 0xffu) * 0xffff0000u);
      w.y &= (((f.x >> 16) & 0xffu) * 0xffffu) | (((f.x >> 24) & 0xffu) * 0xffff0000u);
      w.z &= ((f.y & 0xffu) * 0xffffu) | (((f.y >> 8) & 0xffu) * 0xffff0000u);
      w.w &= (((f.y >> 16) & 0xffu) * 0xffffu) | (((f.y >> 24) & 0xffu) * 0xffff0000u);
      *reinterpret_cast<uint4*>(J.plan + (static_cast<size_t>(b) * d + r) * J.cols + (q << 3)) = w;
    }
  }
  if (kc == 0) return;

  // ascending list of kept columns
  int running = 0;
  for (int q0 = 0; q0 < chunks; q0 += blockDim.x) {
    const int q = q0 + threadIdx.x;
    uint2 f = make_uint2(0u, 0u);
    if (q < chunks) f = *reinterpret_cast<const uint2*>(flags + (q << 3));
    const int mine = __popc(f.x) + __popc(f.y);
    int total;
    int p = running + block_exclusive_scan(mine, s_warp, &total);
    running += total;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const uint32_t bit = ((i < 4 ? f.x : f.y) >> (8 * (i & 3))) & 1u;
      if (bit) s_idx[p++] = (q << 3) + i;
    }
  }
  __syncthreads();
  if (blockIdx.y == 0)
    for (int p = threadIdx.x; p < kc; p += blockDim.x) J.idx[base + p] = s_idx[p];
  uint16_t* tile = J.vals + static_cast<size_t>(d) * base;
  for (int p = threadIdx.x; p < kc; p += blockDim.x) {
    const int col = s_idx[p];
    int r = r_lo;
    for (; r + 4 <= r_hi; r += 4) {
      uint16_t v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) v[u] = __ldg(wblk + static_cast<size_t>(r + u) * J.ldw + col);
#pragma unroll
      for (int u = 0; u < 4; ++u) tile[static_cast<size_t>(r + u) * kc + p] = v[u];
    }
    for (; r < r_hi; ++r) tile[static_cast<size_t>(r) * kc + p] = __ldg(wblk + static_cast<size_t>(r) * J.ldw + col);
  }
}

}  // namespace
}  // namespace bsp

extern "C" int bsp_prepare_batched(const bsp_layer_job* jobs, int n_jobs, int block, float eps, int pen,
                                   void* stream) {
  using namespace bsp;
  if (jobs == nullptr || n_jobs <= 0 || block <= 0) return BSP_ERR_ARG;
  if (pen != BSP_PEN_L2 && pen != BSP_PEN_L2SQ) return BSP_ERR_ARG;
  if (!(eps >= 0.0f)) return BSP_ERR_ARG;
  // validate everything before the first launch
  for (int i = 0; i < n_jobs; ++i) {
    const bsp_layer_job& u = jobs[i];
    int st = check_matrix_args(u.W, u.rows, u.cols, u.ldw, block, BSP_ORIENT_C);
    if (st != BSP_OK) return st;
    if (u.blk_ptr == nullptr || u.idx == nullptr || u.vals == nullptr || u.ws == nullptr) return BSP_ERR_ARG;
    if (!aligned_to(u.ws, 256) || !aligned_to(u.blk_ptr, 4) || !aligned_to(u.idx, 4) || !aligned_to(u.vals, 2)) return BSP_ERR_ARG;
    if (u.threshold != u.threshold) return BSP_ERR_ARG;
    const int nb = u.rows / block;
    if (u.ws_bytes < ws_layout(nb, u.cols).total) return BSP_ERR_WORKSPACE;
    if (u.plan != nullptr) {
      if (!aligned_to(u.plan, 256)) return BSP_ERR_ARG;
      if (u.plan_bytes < static_cast<size_t>(u.rows) * u.cols * 2) return BSP_ERR_WORKSPACE;
    }
    const bool fast = u.cols % 8 == 0 && u.ldw % 8 == 0 && aligned_to(u.W, 16) && u.cols <= 12288 && nb <= 8192 &&
                      (u.keep == nullptr || aligned_to(u.keep, 8)) &&
                      (u.norms == nullptr || aligned_to(u.norms, 4)) && (u.gamma_out == nullptr || aligned_to(u.gamma_out, 4));
    if (!fast) return BSP_ERR_UNSUPPORTED;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  for (int j0 = 0; j0 < n_jobs; j0 += kMaxJobs) {
    Batch B;
    B.n_jobs = n_jobs - j0 < kMaxJobs ? n_jobs - j0 : kMaxJobs;
    B.block = block;
    int total_blocks = 0, max_cols = 0;
    for (int i = 0; i < B.n_jobs; ++i) {
      const bsp_layer_job& u = jobs[j0 + i];
      Job& J = B.job[i];
      const int nb = u.rows / block;
      const WsLayout L = ws_layout(nb, u.cols);
      char* wsb = static_cast<char*>(u.ws);
      J.W = static_cast<const uint16_t*>(u.W);
      J.rows = u.rows; J.cols = u.cols; J.ldw = u.ldw; J.n_blocks = nb;
      J.threshold = u.threshold; J.threshold_dev = u.threshold_dev;
      J.out = NormOut{u.norms, u.gamma_in, u.gamma_out, nullptr, eps, pen == BSP_PEN_L2SQ ? 1 : 0};
      J.penalty = u.penalty;
      J.flags = u.keep ? u.keep : reinterpret_cast<uint8_t*>(wsb + L.keep_off);
      J.counts = reinterpret_cast<int32_t*>(wsb + L.counts_off);
      J.partial = reinterpret_cast<double*>(wsb + L.sumsq_off);
      J.blk_ptr = u.blk_ptr; J.idx = u.idx; J.vals = static_cast<uint16_t*>(u.vals);
      J.kept_weights = u.kept_weights; J.plan = static_cast<uint16_t*>(u.plan);
      B.first_block[i] = total_blocks;
      total_blocks += nb;
      if (u.cols > max_cols) max_cols = u.cols;
    }
    B.first_block[B.n_jobs] = total_blocks;
    fused_norms_flags_kernel<<<total_blocks, kThreads, 0, s>>>(B);
    BSP_LAUNCH_CHECK();
    const int splits = block >= 4 ? 4 : 1;
    fused_compact_plan_kernel<<<dim3(total_blocks, splits), kThreads, sizeof(int32_t) * max_cols, s>>>(B);
    BSP_LAUNCH_CHECK();
  }
  return BSP_OK;
}
