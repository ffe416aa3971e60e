// bsp_prune_pack, bsp_percentile_threshold, bsp_apply_mask: Algorithm 1's keep decision per
// group, Algorithm 2's mask, and the compaction of the kept groups into the canonical
// block-structured storage (Section 3.1).
//
// Launches per pack: (1) one CTA per block decides its groups and counts the kept ones,
// (2) CTAs per block turn the counts before theirs into blk_ptr, list the kept indices in
// ascending order and gather the dense tile of kept values.  W is read from HBM once by (1);
// (2) re-reads it from L2.  Orientation C with 8-element alignment runs the vectorised
// two-stage kernels of bsp_fused.cu; this file holds the generic kernels (any alignment,
// orientation R, with a single-CTA scan between (1) and (2)), the keep-count and percentile
// kernels, and the entry points.
#include <mutex>
#include <new>

#include "bsp_common.cuh"

namespace bsp {
namespace {

constexpr int kPackThreads = 256;

struct Geometry {
  int rows, cols, ldw, block, orient, n_blocks, n_groups;
};

// Pointer to element 0 of group g of block b, and the stride between the group's elements.
__device__ __forceinline__ const uint16_t* group_ptr(const uint16_t* W, const Geometry& G, int b, int g,
                                                     size_t* stride) {
  if (G.orient == BSP_ORIENT_C) {
    *stride = G.ldw;
    return W + static_cast<size_t>(b) * G.block * G.ldw + g;
  }
  *stride = 1;
  return W + static_cast<size_t>(g) * G.ldw + static_cast<size_t>(b) * G.block;
}

// Position of group g of block b in a per-group array ([rows/d, cols] for C, [rows, cols/h] for R).
__device__ __forceinline__ size_t group_slot(const Geometry& G, int b, int g) {
  return G.orient == BSP_ORIENT_C ? static_cast<size_t>(b) * G.n_groups + g
                                  : static_cast<size_t>(g) * G.n_blocks + b;
}

// (1a) threshold mode.
__global__ void __launch_bounds__(kPackThreads)
flags_threshold_kernel(const uint16_t* __restrict__ W, Geometry G, float threshold,
                       const float* __restrict__ threshold_dev, uint8_t* __restrict__ keep,
                       int32_t* __restrict__ counts) {
  __shared__ int s_count;
  if (threadIdx.x == 0) s_count = 0;
  __syncthreads();
  const float t = threshold_dev ? *threshold_dev : threshold;
  const bool keep_all = t < 0.0f;
  const float t2 = __fmul_rn(t, t);
  const int b = blockIdx.x;
  int local = 0;
  for (int g = threadIdx.x; g < G.n_groups; g += blockDim.x) {
    size_t stride;
    const uint16_t* p = group_ptr(W, G, b, g, &stride);
    const float S = group_sumsq_strided(p, G.block, stride);
    const bool k = keep_all || (S > t2);
    keep[group_slot(G, b, g)] = k ? 1 : 0;
    local += k ? 1 : 0;
  }
  local = warp_sum(local);
  if ((threadIdx.x & 31) == 0 && local) atomicAdd(&s_count, local);
  __syncthreads();
  if (threadIdx.x == 0) counts[b] = s_count;
}

// (1b) keep-count mode: rank every group of the block by (larger S first, lower index first).
__global__ void __launch_bounds__(kPackThreads)
flags_topk_kernel(const uint16_t* __restrict__ W, Geometry G, int keep_count,
                  uint8_t* __restrict__ keep, int32_t* __restrict__ counts) {
  extern __shared__ float s_S[];
  const int b = blockIdx.x;
  for (int g = threadIdx.x; g < G.n_groups; g += blockDim.x) {
    size_t stride;
    const uint16_t* p = group_ptr(W, G, b, g, &stride);
    s_S[g] = group_sumsq_strided(p, G.block, stride);
  }
  __syncthreads();
  for (int g = threadIdx.x; g < G.n_groups; g += blockDim.x) {
    const float mine = s_S[g];
    int rank = 0;
    for (int o = 0; o < G.n_groups; ++o) {
      const float other = s_S[o];
      rank += (other > mine || (other == mine && o < g)) ? 1 : 0;
    }
    keep[group_slot(G, b, g)] = rank < keep_count ? 1 : 0;
  }
  if (threadIdx.x == 0) counts[b] = keep_count < G.n_groups ? keep_count : G.n_groups;
}

// (2) counts -> blk_ptr (exclusive scan) and the kept-weight total.
__global__ void __launch_bounds__(1024)
scan_counts_kernel(const int32_t* __restrict__ counts, int n_blocks, int block,
                   int32_t* __restrict__ blk_ptr, int64_t* __restrict__ kept_weights) {
  __shared__ int s_warp[32];
  int running = 0;
  for (int base = 0; base < n_blocks; base += blockDim.x) {
    const int i = base + threadIdx.x;
    const int v = i < n_blocks ? counts[i] : 0;
    int total;
    const int excl = block_exclusive_scan(v, s_warp, &total);
    if (i < n_blocks) blk_ptr[i] = running + excl;
    running += total;
  }
  if (threadIdx.x == 0) {
    blk_ptr[n_blocks] = running;
    if (kept_weights) *kept_weights = static_cast<int64_t>(running) * block;
  }
}

// (3) compaction: ascending index list and the dense tile of kept values of one block.
__global__ void __launch_bounds__(kPackThreads)
compact_kernel(const uint16_t* __restrict__ W, Geometry G, const uint8_t* __restrict__ keep,
               const int32_t* __restrict__ blk_ptr, int32_t* __restrict__ idx,
               uint16_t* __restrict__ vals) {
  __shared__ int s_warp[32];
  const int b = blockIdx.x;
  const int base = blk_ptr[b];
  const int kc = blk_ptr[b + 1] - base;
  if (kc == 0) return;
  uint16_t* tile = vals + static_cast<size_t>(G.block) * base;
  int running = 0;
  for (int g0 = 0; g0 < G.n_groups; g0 += blockDim.x) {
    const int g = g0 + threadIdx.x;
    const int k = (g < G.n_groups) ? keep[group_slot(G, b, g)] : 0;
    int total;
    const int p = running + block_exclusive_scan(k, s_warp, &total);
    running += total;
    if (k) {
      idx[base + p] = g;
      size_t stride;
      const uint16_t* src = group_ptr(W, G, b, g, &stride);
      if (G.orient == BSP_ORIENT_C) {
        // tile [d, kc]: element r of the group goes to row r, position p
        for (int r = 0; r < G.block; ++r) tile[static_cast<size_t>(r) * kc + p] = src[static_cast<size_t>(r) * stride];
      } else {
        // tile [kc, h]: the group's h contiguous elements form row p
        for (int c = 0; c < G.block; ++c) tile[static_cast<size_t>(p) * G.block + c] = src[c];
      }
    }
  }
}


// Float32 sums of squares of all groups, flattened in per-group-array order.
__global__ void __launch_bounds__(kPackThreads)
sumsq_kernel(const uint16_t* __restrict__ W, Geometry G, float* __restrict__ S) {
  const int b = blockIdx.x;
  for (int g = threadIdx.x; g < G.n_groups; g += blockDim.x) {
    size_t stride;
    const uint16_t* p = group_ptr(W, G, b, g, &stride);
    S[group_slot(G, b, g)] = group_sumsq_strided(p, G.block, stride);
  }
}

// r-th smallest (1-based) of n non-negative floats by a 4-pass radix select on their bit
// patterns (monotone for non-negative floats), one CTA of 1024 threads; then the threshold whose
// float32 square is >= that value.  Sums of squares of one matrix share their leading byte, so a
// single shared histogram would serialise on two or three counters: every warp counts into its own
// 256-bin histogram and the lanes of a warp that hit the same bin add once (match_any).
__device__ void select_threshold(const float* __restrict__ S, long long n, long long r, float* __restrict__ out,
                                 unsigned int (*hist)[256], unsigned int* s_prefix, long long* s_remaining) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
  if (r <= 0) {
    if (threadIdx.x == 0) *out = -1.0f;
    return;
  }
  if (threadIdx.x == 0) { *s_prefix = 0u; *s_remaining = r; }
  for (int pass = 3; pass >= 0; --pass) {
    for (int i = lane; i < 256; i += 32) hist[warp][i] = 0u;
    __syncthreads();
    const unsigned int prefix = *s_prefix;
    const int shift = pass * 8;
    const unsigned int high_mask = pass == 3 ? 0u : (0xffffffffu << (shift + 8));
    for (long long i0 = 0; i0 < n; i0 += blockDim.x) {
      const long long i = i0 + threadIdx.x;
      unsigned int bin = 0xffffffffu;                    // lanes without an element, or outside the prefix, sit out
      if (i < n) {
        const unsigned int u = __float_as_uint(S[i]);
        if ((u & high_mask) == prefix) bin = (u >> shift) & 0xffu;
      }
      const unsigned int peers = __match_any_sync(0xffffffffu, bin);
      if (bin != 0xffffffffu && lane == __ffs(peers) - 1) hist[warp][bin] += static_cast<unsigned int>(__popc(peers));
    }
    __syncthreads();
    if (threadIdx.x < 256) {                             // fold the warps' histograms into the first one
      unsigned int c = 0;
      for (int w = 0; w < n_warps; ++w) c += hist[w][threadIdx.x];
      hist[0][threadIdx.x] = c;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      long long rem = *s_remaining;
      unsigned int d = 0;
      for (; d < 256; ++d) {
        if (rem <= static_cast<long long>(hist[0][d])) break;
        rem -= hist[0][d];
      }
      *s_prefix = prefix | (d << shift);
      *s_remaining = rem;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const float s_r = __uint_as_float(*s_prefix);
    float t = __fsqrt_rn(s_r);
    while (__fmul_rn(t, t) < s_r) t = __uint_as_float(__float_as_uint(t) + 1u);  // next float up (t >= 0)
    *out = t;
  }
}

__global__ void __launch_bounds__(1024)
select_threshold_kernel(const float* __restrict__ S, long long n, long long r, float* __restrict__ out) {
  __shared__ unsigned int hist[32][256];
  __shared__ unsigned int s_prefix;
  __shared__ long long s_remaining;
  select_threshold(S, n, r, out, hist, &s_prefix, &s_remaining);
}

// The same for a batch of matrices: sums of squares of every row-block of every matrix in one launch
// (orientation C, one CTA per row-block), then one selecting CTA per matrix.
constexpr int kSelectBatch = 96;
struct SelectJob {
  const uint16_t* W;
  int cols, ldw, n_blocks, first_block;
  float* S;
  float* out;
  long long n, r;
};
struct SelectBatch {
  int n_jobs, block;
  SelectJob job[kSelectBatch];
};
__global__ void __launch_bounds__(kPackThreads)
sumsq_batched_kernel(const __grid_constant__ SelectBatch B) {
  int lo = 0, hi = B.n_jobs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (B.job[mid].first_block <= static_cast<int>(blockIdx.x)) lo = mid; else hi = mid - 1;
  }
  const SelectJob& J = B.job[lo];
  const int b = static_cast<int>(blockIdx.x) - J.first_block;
  const uint16_t* wblk = J.W + static_cast<size_t>(b) * B.block * J.ldw;
  for (int g = threadIdx.x; g < J.cols; g += blockDim.x)
    J.S[static_cast<size_t>(b) * J.cols + g] = group_sumsq_strided(wblk + g, B.block, J.ldw);
}
__global__ void __launch_bounds__(1024)
select_threshold_batched_kernel(const __grid_constant__ SelectBatch B) {
  __shared__ unsigned int hist[32][256];
  __shared__ unsigned int s_prefix;
  __shared__ long long s_remaining;
  const SelectJob& J = B.job[blockIdx.x];
  select_threshold(J.S, J.n, J.r, J.out, hist, &s_prefix, &s_remaining);
}

__global__ void __launch_bounds__(256)
apply_mask_kernel(uint16_t* __restrict__ W, Geometry G, const uint8_t* __restrict__ keep) {
  const long long e = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (e >= static_cast<long long>(G.rows) * G.cols) return;
  const int i = static_cast<int>(e / G.cols), j = static_cast<int>(e - static_cast<long long>(i) * G.cols);
  const size_t slot = G.orient == BSP_ORIENT_C ? static_cast<size_t>(i / G.block) * G.cols + j
                                               : static_cast<size_t>(i) * (G.cols / G.block) + j / G.block;
  if (!keep[slot]) W[static_cast<size_t>(i) * G.ldw + j] = 0;
}

// Fixed scratch for bsp_prune_pack_static: lives in the library's device image, so every GPU
// that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_pack_scratch[BSP_STATIC_SCRATCH_BYTES];

}  // namespace
}  // namespace bsp

extern "C" int bsp_pack_bound(int rows, int cols, int block, int orient, size_t* idx_elems,
                              size_t* val_elems, size_t* ws_bytes) {
  using namespace bsp;
  if (rows <= 0 || cols <= 0 || block <= 0) return BSP_ERR_ARG;
  if (orient != BSP_ORIENT_C && orient != BSP_ORIENT_R) return BSP_ERR_ARG;
  int nb, ng;
  if (!geometry(rows, cols, block, orient, &nb, &ng)) return BSP_ERR_SHAPE;
  if (idx_elems) *idx_elems = static_cast<size_t>(nb) * ng;
  if (val_elems) *val_elems = static_cast<size_t>(rows) * cols;
  if (ws_bytes) *ws_bytes = ws_layout(nb, ng).total;
  return BSP_OK;
}

extern "C" int bsp_pack_scratch_bytes(int rows, int cols, int block, int orient, size_t* bytes) {
  using namespace bsp;
  if (rows <= 0 || cols <= 0 || block <= 0 || bytes == nullptr) return BSP_ERR_ARG;
  if (orient != BSP_ORIENT_C && orient != BSP_ORIENT_R) return BSP_ERR_ARG;
  int nb, ng;
  if (!geometry(rows, cols, block, orient, &nb, &ng)) return BSP_ERR_SHAPE;
  *bytes = ws_layout(nb, ng).sumsq_off;
  return BSP_OK;
}

extern "C" int bsp_prune_pack(const void* W, int rows, int cols, int ldw, int block, int orient,
                              float threshold, const float* threshold_dev, int keep_per_block,
                              uint8_t* keep, int32_t* blk_ptr, int32_t* idx, void* vals,
                              int64_t* kept_weights, void* ws, size_t ws_bytes, void* stream) {
  using namespace bsp;
  int st = check_matrix_args(W, rows, cols, ldw, block, orient);
  if (st != BSP_OK) return st;
  if (blk_ptr == nullptr || idx == nullptr || vals == nullptr || ws == nullptr) return BSP_ERR_ARG;
  if (!aligned_to(ws, 256) || !aligned_to(vals, 2) || !aligned_to(blk_ptr, 4) || !aligned_to(idx, 4)) return BSP_ERR_ARG;
  if (threshold != threshold) return BSP_ERR_ARG;  // NaN
  Geometry G{rows, cols, ldw, block, orient, 0, 0};
  geometry(rows, cols, block, orient, &G.n_blocks, &G.n_groups);
  const WsLayout L = ws_layout(G.n_blocks, G.n_groups);
  if (ws_bytes < L.sumsq_off) return BSP_ERR_WORKSPACE;   // counts and flags; the float32 region is the percentile call's
  if (keep_per_block >= 0 && G.n_groups > BSP_TOPK_MAX_GROUPS) return BSP_ERR_UNSUPPORTED;

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* wsb = static_cast<char*>(ws);
  int32_t* counts = reinterpret_cast<int32_t*>(wsb + L.counts_off);
  uint8_t* flags = keep ? keep : reinterpret_cast<uint8_t*>(wsb + L.keep_off);
  const uint16_t* w = static_cast<const uint16_t*>(W);

  const bool fast = orient == BSP_ORIENT_C && fused_shape_ok(W, rows, cols, ldw, block) && aligned_to(flags, 8);
  if (fast) {
    // vectorised kernels of bsp_fused.cu: stage 1 for the flags (unless the keep-count kernel makes them), stage 2
    FusedJob j{w, rows, cols, ldw, G.n_blocks, threshold, threshold_dev, nullptr, nullptr, nullptr, nullptr, nullptr,
               flags, counts, blk_ptr, idx, static_cast<uint16_t*>(vals), kept_weights, nullptr};
    if (keep_per_block >= 0) {
      flags_topk_kernel<<<G.n_blocks, kPackThreads, sizeof(float) * G.n_groups, s>>>(w, G, keep_per_block, flags, counts);
      BSP_LAUNCH_CHECK();
    } else {
      st = fused_stage1(&j, 1, block, 0.0f, 0, s);
      if (st != BSP_OK) return st;
    }
    return fused_stage2(&j, 1, block, s);
  }
  if (keep_per_block >= 0) {
    flags_topk_kernel<<<G.n_blocks, kPackThreads, sizeof(float) * G.n_groups, s>>>(w, G, keep_per_block, flags, counts);
  } else {
    flags_threshold_kernel<<<G.n_blocks, kPackThreads, 0, s>>>(w, G, threshold, threshold_dev, flags, counts);
  }
  BSP_LAUNCH_CHECK();
  scan_counts_kernel<<<1, 1024, 0, s>>>(counts, G.n_blocks, block, blk_ptr, kept_weights);
  BSP_LAUNCH_CHECK();
  compact_kernel<<<G.n_blocks, kPackThreads, 0, s>>>(w, G, flags, blk_ptr, idx, static_cast<uint16_t*>(vals));
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

extern "C" int bsp_percentile_threshold(const void* W, int rows, int cols, int ldw, int block,
                                        int orient, double rate, float* threshold_out, void* ws,
                                        size_t ws_bytes, void* stream) {
  using namespace bsp;
  int st = check_matrix_args(W, rows, cols, ldw, block, orient);
  if (st != BSP_OK) return st;
  if (threshold_out == nullptr || ws == nullptr || !aligned_to(ws, 256)) return BSP_ERR_ARG;
  if (!(rate >= 1.0)) return BSP_ERR_ARG;
  Geometry G{rows, cols, ldw, block, orient, 0, 0};
  geometry(rows, cols, block, orient, &G.n_blocks, &G.n_groups);
  const WsLayout L = ws_layout(G.n_blocks, G.n_groups);
  if (ws_bytes < L.total) return BSP_ERR_WORKSPACE;
  const long long groups = static_cast<long long>(G.n_blocks) * G.n_groups;
  // r = floor(G * (1 - 1/c)) in float64, as the definition states it
  const long long r = static_cast<long long>(static_cast<double>(groups) * (1.0 - 1.0 / rate));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  float* S = reinterpret_cast<float*>(static_cast<char*>(ws) + L.sumsq_off);
  sumsq_kernel<<<G.n_blocks, kPackThreads, 0, s>>>(static_cast<const uint16_t*>(W), G, S);
  BSP_LAUNCH_CHECK();
  select_threshold_kernel<<<1, 1024, 0, s>>>(S, groups, r, threshold_out);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

extern "C" int bsp_percentile_threshold_batched(const bsp_layer_job* jobs, int n_jobs, int block, const double* rates,
                                                void* stream) {
  using namespace bsp;
  if (jobs == nullptr || rates == nullptr || n_jobs <= 0 || block <= 0) return BSP_ERR_ARG;
  if (n_jobs > 4096) return BSP_ERR_UNSUPPORTED;
  for (int i = 0; i < n_jobs; ++i) {                       // everything is checked before the first launch
    const bsp_layer_job& u = jobs[i];
    int st = check_matrix_args(u.W, u.rows, u.cols, u.ldw, block, BSP_ORIENT_C);
    if (st != BSP_OK) return st;
    if (u.threshold_dev == nullptr || u.ws == nullptr || !aligned_to(u.ws, 256)) return BSP_ERR_ARG;
    if (!(rates[i] >= 1.0)) return BSP_ERR_ARG;
    if (u.ws_bytes < ws_layout(u.rows / block, u.cols).total) return BSP_ERR_WORKSPACE;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  SelectBatch* B = new (std::nothrow) SelectBatch;
  if (B == nullptr) return BSP_ERR_ARG;
  int st = BSP_OK;
  for (int j0 = 0; j0 < n_jobs && st == BSP_OK; j0 += kSelectBatch) {
    const int n = n_jobs - j0 < kSelectBatch ? n_jobs - j0 : kSelectBatch;
    B->n_jobs = n;
    B->block = block;
    int blocks = 0;
    for (int i = 0; i < n; ++i) {
      const bsp_layer_job& u = jobs[j0 + i];
      const int nb = u.rows / block;
      const long long groups = static_cast<long long>(nb) * u.cols;
      SelectJob& J = B->job[i];
      J.W = static_cast<const uint16_t*>(u.W);
      J.cols = u.cols;
      J.ldw = u.ldw;
      J.n_blocks = nb;
      J.first_block = blocks;
      J.S = reinterpret_cast<float*>(static_cast<char*>(u.ws) + ws_layout(nb, u.cols).sumsq_off);
      J.out = const_cast<float*>(u.threshold_dev);
      J.n = groups;
      J.r = static_cast<long long>(static_cast<double>(groups) * (1.0 - 1.0 / rates[j0 + i]));   // as the single-matrix call
      blocks += nb;
    }
    sumsq_batched_kernel<<<blocks, kPackThreads, 0, s>>>(*B);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) {
      select_threshold_batched_kernel<<<n, 1024, 0, s>>>(*B);
      e = cudaGetLastError();
    }
    if (e != cudaSuccess) st = cuda_fail(e);
  }
  delete B;
  return st;
}

extern "C" int bsp_apply_mask(void* W, int rows, int cols, int ldw, int block, int orient,
                              const uint8_t* keep, void* stream) {
  using namespace bsp;
  int st = check_matrix_args(W, rows, cols, ldw, block, orient);
  if (st != BSP_OK) return st;
  if (keep == nullptr) return BSP_ERR_ARG;
  Geometry G{rows, cols, ldw, block, orient, 0, 0};
  geometry(rows, cols, block, orient, &G.n_blocks, &G.n_groups);
  const long long elems = static_cast<long long>(rows) * cols;
  apply_mask_kernel<<<static_cast<unsigned>((elems + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<uint16_t*>(W), G, keep);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

extern "C" int bsp_prune_pack_static(const void* W, int rows, int cols, int ldw, int block, int orient,
                                     float threshold, const float* threshold_dev, int keep_per_block,
                                     uint8_t* keep, int32_t* blk_ptr, int32_t* idx, void* vals,
                                     int64_t* kept_weights, void* stream) {
  using namespace bsp;
  int st = check_matrix_args(W, rows, cols, ldw, block, orient);
  if (st != BSP_OK) return st;
  size_t need = 0;
  st = bsp_pack_scratch_bytes(rows, cols, block, orient, &need);
  if (st != BSP_OK) return st;
  if (need > static_cast<size_t>(BSP_STATIC_SCRATCH_BYTES)) return BSP_ERR_UNSUPPORTED;

  // In host code the array's name is only a handle; the device address has to be asked for,
  // once per device, while that device is current.
  static void* scratch_of_device[64] = {nullptr};
  static std::mutex guard;
  std::lock_guard<std::mutex> lock(guard);
  int dev = -1;
  BSP_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return BSP_ERR_UNSUPPORTED;
  if (scratch_of_device[dev] == nullptr) {
    void* ptr = nullptr;
    BSP_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_pack_scratch));
    if (ptr == nullptr) return BSP_ERR_CUDA;
    scratch_of_device[dev] = ptr;
  }
  // Every byte of the scratch that the kernels read (per-block counts, per-group flags) is
  // written earlier in the same call, so nothing left over from the previous call is observed
  // and nothing needs clearing.
  return bsp_prune_pack(W, rows, cols, ldw, block, orient, threshold, threshold_dev, keep_per_block, keep, blk_ptr,
                        idx, vals, kept_weights, scratch_of_device[dev], BSP_STATIC_SCRATCH_BYTES, stream);
}
