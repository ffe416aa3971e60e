// One-launch variant of the vectorised weight-side kernels, for batches small enough that all of
// their CTAs are resident at once (the four matrices of an encoder layer, say).
//
// The two-stage kernels of bsp_fused.cu read W twice and pay two launches; at a few megabytes both
// launches are pure latency.  Here a CTA owns one row-block of one matrix (or a column range of it,
// so that its rows fit 32 KB of shared memory), loads those rows ONCE into shared memory, and
//   phase A  computes the float32 sums of squares from shared memory (rows in increasing order, the
//            defined decision quantity), writes norms / gamma / keep flags, and publishes its kept
//            count and penalty partial;
//   -- cooperative grid barrier --
//   phase B  sums the counts published before it (blk_ptr), lists its kept columns, and writes its
//            part of the packed tile and of the zero-expanded execution layout from shared memory.
// Masks, indices, tiles, norms and gamma are bit-identical to the two-stage path; the penalty is
// the same up to its (fixed, reproducible) summation order.
#include <cooperative_groups.h>

#include "bsp_common.cuh"

namespace cg = cooperative_groups;

namespace bsp {
namespace {

constexpr int kOneMaxJobs = 16;
constexpr int kOneThreads = 256;
constexpr int kOneRowBytes = 32 * 1024;     // shared memory for a CTA's rows

struct OneJob {
  FusedJob j;
  int parts, part_cols;      // column ranges per row-block, columns per range (multiple of 8)
  int first_cta;
  int32_t* part_counts;      // [n_blocks][parts]
  double* part_partial;      // [n_blocks][parts]
};
struct OneBatch {
  int n_jobs, block, squared;
  float eps;
  OneJob job[kOneMaxJobs];
};

__global__ void __launch_bounds__(kOneThreads)
fused_onepass_kernel(const __grid_constant__ OneBatch B) {
  extern __shared__ __align__(16) uint8_t s_raw[];
  __shared__ int s_cnt[8];
  __shared__ double s_pen[8];
  __shared__ int s_warp[32];
  __shared__ int s_sum[2];
  int jn = 0;
  while (jn + 1 < B.n_jobs && static_cast<int>(blockIdx.x) >= B.job[jn + 1].first_cta) ++jn;
  const OneJob& O = B.job[jn];
  const FusedJob& J = O.j;
  const int local = blockIdx.x - O.first_cta;
  const int b = local / O.parts, q = local - b * O.parts;
  const int d = B.block;
  const int c0 = q * O.part_cols;
  const int pc = min(O.part_cols, J.cols - c0);          // columns of this CTA (multiple of 8)
  const int chunks = pc >> 3;
  uint16_t* s_w = reinterpret_cast<uint16_t*>(s_raw);                                  // [d][pc]
  int32_t* s_idx = reinterpret_cast<int32_t*>(s_raw + static_cast<size_t>(d) * O.part_cols * 2);   // [pc]
  uint8_t* s_flag = reinterpret_cast<uint8_t*>(s_idx + O.part_cols);                   // [pc]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
  const uint16_t* wblk = J.W + static_cast<size_t>(b) * d * J.ldw + c0;

  // ---- rows of this CTA into shared memory: one warp per row, 16-byte loads, four in flight per lane
  for (int r = warp; r < d; r += n_warps) {
    const uint16_t* src = wblk + static_cast<size_t>(r) * J.ldw;
    for (int k0 = lane; k0 < chunks; k0 += 128) {
      uint4 w[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (k0 + 32 * u < chunks) w[u] = __ldg(reinterpret_cast<const uint4*>(src + ((k0 + 32 * u) << 3)));
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (k0 + 32 * u < chunks) *reinterpret_cast<uint4*>(s_w + r * pc + ((k0 + 32 * u) << 3)) = w[u];
    }
  }
  __syncthreads();

  // ---- phase A: sums of squares of 8 adjacent columns per thread, rows in increasing order
  const bool want_pen = J.penalty != nullptr;
  const bool want_norms = J.norms != nullptr || J.gamma_out != nullptr || want_pen;
  const float t = J.threshold_dev ? *J.threshold_dev : J.threshold;
  const bool keep_all = t < 0.0f;
  const float t2 = __fmul_rn(t, t);
  int count = 0;
  float pen = 0.0f;
  for (int k = threadIdx.x; k < chunks; k += blockDim.x) {
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.0f;
    for (int r = 0; r < d; ++r) {
      const uint4 v = *reinterpret_cast<const uint4*>(s_w + r * pc + (k << 3));
      const uint32_t w32[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float lo = __uint_as_float(w32[i] << 16), hi = __uint_as_float(w32[i] & 0xffff0000u);
        acc[2 * i] = __fmaf_rn(lo, lo, acc[2 * i]);
        acc[2 * i + 1] = __fmaf_rn(hi, hi, acc[2 * i + 1]);
      }
    }
    uint32_t lo = 0, hi = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t k0 = (keep_all || acc[i] > t2) ? 1u : 0u;
      const uint32_t k1 = (keep_all || acc[4 + i] > t2) ? 1u : 0u;
      lo |= k0 << (8 * i);
      hi |= k1 << (8 * i);
      count += static_cast<int>(k0 + k1);
    }
    const size_t g0 = static_cast<size_t>(b) * J.cols + c0 + (k << 3);
    *reinterpret_cast<uint2*>(s_flag + (k << 3)) = make_uint2(lo, hi);
    *reinterpret_cast<uint2*>(J.flags + g0) = make_uint2(lo, hi);
    if (want_norms) {
      float n[8], base[8], fresh[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        n[i] = __fsqrt_rn(acc[i]);
        base[i] = B.squared ? acc[i] : n[i];
        fresh[i] = __fdiv_rn(1.0f, base[i] + B.eps);
      }
      if (J.norms) {
        *reinterpret_cast<float4*>(J.norms + g0) = make_float4(n[0], n[1], n[2], n[3]);
        *reinterpret_cast<float4*>(J.norms + g0 + 4) = make_float4(n[4], n[5], n[6], n[7]);
      }
      if (J.gamma_out) {
        *reinterpret_cast<float4*>(J.gamma_out + g0) = make_float4(fresh[0], fresh[1], fresh[2], fresh[3]);
        *reinterpret_cast<float4*>(J.gamma_out + g0 + 4) = make_float4(fresh[4], fresh[5], fresh[6], fresh[7]);
      }
      if (want_pen) {
        if (J.gamma_in) {
          const float4 a = __ldg(reinterpret_cast<const float4*>(J.gamma_in + g0));
          const float4 c = __ldg(reinterpret_cast<const float4*>(J.gamma_in + g0 + 4));
          const float w[8] = {a.x, a.y, a.z, a.w, c.x, c.y, c.z, c.w};
#pragma unroll
          for (int i = 0; i < 8; ++i) pen = fmaf(w[i], base[i], pen);
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) pen = fmaf(fresh[i], base[i], pen);
        }
      }
    }
  }
  count = warp_sum(count);
  double pd = warp_sum(static_cast<double>(pen));
  if (lane == 0) { s_cnt[warp] = count; s_pen[warp] = pd; }
  __syncthreads();
  if (threadIdx.x == 0) {
    int c = 0;
    double p = 0.0;
    for (int w = 0; w < n_warps; ++w) { c += s_cnt[w]; p += s_pen[w]; }
    O.part_counts[local] = c;
    O.part_partial[local] = p;
  }

  cg::this_grid().sync();      // every CTA's count and partial are published

  // ---- phase B: offsets from the published counts
  // kept groups of this matrix before this CTA's (block, part), and within its block
  int before = 0, in_block_before = 0, in_block = 0;
  for (int i = threadIdx.x; i < local; i += blockDim.x) before += O.part_counts[i];
  for (int i = threadIdx.x; i < O.parts; i += blockDim.x) {
    const int c = O.part_counts[b * O.parts + i];
    in_block += c;
    if (i < q) in_block_before += c;
  }
  before = warp_sum(before);
  in_block = warp_sum(in_block);
  in_block_before = warp_sum(in_block_before);
  if (threadIdx.x == 0) { s_sum[0] = 0; s_sum[1] = 0; }
  __syncthreads();
  if (lane == 0) {
    if (before) atomicAdd(&s_sum[0], before);
    if (in_block) atomicAdd(&s_sum[1], in_block);
  }
  // in_block_before: only the first min(parts, blockDim) threads contribute; parts <= 32 keeps it in warp 0
  __shared__ int s_inb;
  if (threadIdx.x == 0) s_inb = 0;
  __syncthreads();
  if (lane == 0 && in_block_before) atomicAdd(&s_inb, in_block_before);
  __syncthreads();
  const int base = s_sum[0];               // kept groups before this CTA's first one (index into idx)
  const int kc_block = s_sum[1];           // kept groups of the whole row-block
  const int off_in_block = s_inb;          // kept groups of the block's earlier parts
  const int kc = O.part_counts[local];     // kept groups of this part
  const int block_base = base - off_in_block;
  if (q == 0 && threadIdx.x == 0) {
    J.blk_ptr[b] = block_base;
    if (b == J.n_blocks - 1) {
      J.blk_ptr[J.n_blocks] = block_base + kc_block;
      if (J.kept_weights) *J.kept_weights = static_cast<int64_t>(block_base + kc_block) * d;
    }
  }
  // penalty total of the job, by its first CTA, in a fixed order
  if (local == 0 && J.penalty != nullptr) {
    double p = 0.0;
    const int n_parts = J.n_blocks * O.parts;
    for (int i = threadIdx.x; i < n_parts; i += blockDim.x) p += O.part_partial[i];
    p = warp_sum(p);
    __syncthreads();
    if (lane == 0) s_pen[warp] = p;
    __syncthreads();
    if (threadIdx.x == 0) {
      double tot = 0.0;
      for (int w = 0; w < n_warps; ++w) tot += s_pen[w];
      *J.penalty = tot;
    }
  }

  // execution layout: the rows with the pruned columns zeroed, one warp per row, 16-byte stores
  if (J.plan != nullptr) {
    for (int r = warp; r < d; r += n_warps) {
      uint16_t* pdst = J.plan + (static_cast<size_t>(b) * d + r) * J.cols + c0;
      for (int k = lane; k < chunks; k += 32) {
        const uint4 w = *reinterpret_cast<const uint4*>(s_w + r * pc + (k << 3));
        const uint2 f = *reinterpret_cast<const uint2*>(s_flag + (k << 3));
        uint4 m;   // a flag byte is 0 or 1: flag * 0xffff masks the matching 16-bit element
        m.x = w.x & (((f.x & 0xffu) * 0xffffu) | (((f.x >> 8) & 0xffu) * 0xffff0000u));
        m.y = w.y & ((((f.x >> 16) & 0xffu) * 0xffffu) | (((f.x >> 24) & 0xffu) * 0xffff0000u));
        m.z = w.z & (((f.y & 0xffu) * 0xffffu) | (((f.y >> 8) & 0xffu) * 0xffff0000u));
        m.w = w.w & ((((f.y >> 16) & 0xffu) * 0xffffu) | (((f.y >> 24) & 0xffu) * 0xffff0000u));
        *reinterpret_cast<uint4*>(pdst + (k << 3)) = m;
      }
    }
  }
  if (kc == 0) return;

  // ascending list of this part's kept columns (local indices in s_idx, global ones to idx)
  int running = 0;
  for (int k0 = 0; k0 < chunks; k0 += blockDim.x) {
    const int k = k0 + threadIdx.x;
    uint2 f = make_uint2(0u, 0u);
    if (k < chunks) f = *reinterpret_cast<const uint2*>(s_flag + (k << 3));
    const int mine = __popc(f.x) + __popc(f.y);
    int total;
    int p = running + block_exclusive_scan(mine, s_warp, &total);
    running += total;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const uint32_t bit = ((i < 4 ? f.x : f.y) >> (8 * (i & 3))) & 1u;
      if (bit) s_idx[p++] = (k << 3) + i;
    }
  }
  __syncthreads();
  for (int p = threadIdx.x; p < kc; p += blockDim.x) J.idx[base + p] = c0 + s_idx[p];

  // packed tile: row r of the block occupies vals[tile0 + r*kc_block, +kc_block); this part fills
  // positions [off_in_block, off_in_block + kc) of every row.  One warp per row; whole 16-byte
  // vectors where the destination is aligned, ragged ends by element.
  const bool vec_ok = (reinterpret_cast<uintptr_t>(J.vals) & 15) == 0;
  const long long tile0 = static_cast<long long>(d) * block_base;
  for (int r = warp; r < d; r += n_warps) {
    const uint16_t* srow = s_w + r * pc;
    const long long e0 = tile0 + static_cast<long long>(r) * kc_block + off_in_block;
    uint16_t* out_row = J.vals + e0;
    if (vec_ok) {
      const int head = static_cast<int>((8 - (e0 & 7)) & 7);
      const int n_vec = kc > head ? (kc - head) >> 3 : 0;
      for (int v = lane; v < n_vec; v += 32) {
        const int p = head + (v << 3);
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
          o[i] = static_cast<uint32_t>(srow[s_idx[p + 2 * i]]) | (static_cast<uint32_t>(srow[s_idx[p + 2 * i + 1]]) << 16);
        *reinterpret_cast<uint4*>(out_row + p) = make_uint4(o[0], o[1], o[2], o[3]);
      }
      const int tail0 = head + (n_vec << 3);
      if (lane < 8) {
        if (lane < head && lane < kc) out_row[lane] = srow[s_idx[lane]];
      } else if (lane < 16) {
        const int p = tail0 + (lane - 8);
        if (p >= head && p < kc) out_row[p] = srow[s_idx[p]];
      }
    } else {
      for (int p = lane; p < kc; p += 32) out_row[p] = srow[s_idx[p]];
    }
  }
}

}  // namespace

// Runs the batch in one cooperative launch if every CTA can be resident at once; *used tells the
// caller whether it did (otherwise nothing was launched and the two-stage path should run).
int fused_onepass(const FusedJob* jobs, int n_jobs, int block, float eps, int squared, int32_t* const* part_counts,
                  double* const* part_partial, cudaStream_t s, bool* used) {
  *used = false;
  if (n_jobs > kOneMaxJobs) return BSP_OK;
  OneBatch B;
  B.n_jobs = n_jobs;
  B.block = block;
  B.squared = squared;
  B.eps = eps;
  int total = 0, max_part_cols = 0;
  for (int i = 0; i < n_jobs; ++i) {
    OneJob& O = B.job[i];
    O.j = jobs[i];
    const int cols = jobs[i].cols;
    int max_cols = (kOneRowBytes / (2 * block)) / 8 * 8;        // columns whose rows fit the row buffer
    if (max_cols < 8) return BSP_OK;
    O.parts = (cols + max_cols - 1) / max_cols;
    O.part_cols = ((cols + O.parts - 1) / O.parts + 7) / 8 * 8;
    O.parts = (cols + O.part_cols - 1) / O.part_cols;
    if (O.parts > 32) return BSP_OK;
    O.first_cta = total;
    O.part_counts = part_counts[i];
    O.part_partial = part_partial[i];
    total += jobs[i].n_blocks * O.parts;
    if (O.part_cols > max_part_cols) max_part_cols = O.part_cols;
  }
  const size_t smem = static_cast<size_t>(max_part_cols) * (2 * block + 4 + 1) + 16;
  if (smem > 48 * 1024) return BSP_OK;
  int dev = 0;
  BSP_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return BSP_OK;
  int per_sm = 0, sms = 0;
  BSP_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fused_onepass_kernel, kOneThreads, smem));
  BSP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  if (total > per_sm * sms) return BSP_OK;

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(total);
  cfg.blockDim = dim3(kOneThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  BSP_CUDA_TRY(cudaLaunchKernelEx(&cfg, fused_onepass_kernel, B));
  *used = true;
  return BSP_OK;
}

}  // namespace bsp
