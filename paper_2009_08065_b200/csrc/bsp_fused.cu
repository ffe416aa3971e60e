// Vectorised orientation-C kernels shared by bsp_group_norms, bsp_prune_pack and
// bsp_prepare_batched.  Two stages over a batch of matrices:
//   stage 1  one CTA per row-block, one thread per 8 adjacent columns: 16-byte loads down the
//            block's rows (8 rows in flight), eight independent sequential float32 sums of
//            squares (the defined decision quantity), then any of: norms / gamma (two 16-byte
//            stores each), penalty partial, keep flags (one 8-byte store) and the block's count.
//   stage 2  grid (row-blocks, row ranges of about 16K weights): blk_ptr from the counts before
//            the block, the ascending index list from the flags, then 4 rows at a time staged in
//            shared memory (16-byte loads) and from there (a) the zero-expanded execution
//            layout, (b) the packed tile, written as 16-byte vectors wherever the output is
//            16-byte aligned.
#include <new>

#include "bsp_common.cuh"

namespace bsp {
namespace {

constexpr int kRowsPerPass = 4;   // rows staged in shared memory at a time

struct Batch {
  int n_jobs, block, squared;
  float eps;
  int first_block[kFusedMaxJobs + 1];   // CTA index of each job's first row-block
  FusedJob job[kFusedMaxJobs];
};

// Job that owns CTA `cta`: the last j with first_block[j] <= cta (binary search).
__device__ __forceinline__ int find_job(const Batch& B, int cta) {
  int lo = 0, hi = B.n_jobs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (B.first_block[mid] <= cta) lo = mid; else hi = mid - 1;
  }
  return lo;
}

__global__ void __launch_bounds__(256)
fused_stage1_kernel(const __grid_constant__ Batch B) {
  __shared__ int s_cnt[8];
  __shared__ double s_pen[8];
  const int j = find_job(B, blockIdx.x);
  const FusedJob& J = B.job[j];
  const int b = blockIdx.x - B.first_block[j];
  const bool want_flags = J.flags != nullptr;
  const bool want_pen = J.penalty != nullptr;
  const bool want_norms = J.norms != nullptr || J.gamma_out != nullptr || want_pen;
  float t2 = 0.0f;
  bool keep_all = false;
  if (want_flags) {
    const float t = J.threshold_dev ? *J.threshold_dev : J.threshold;
    keep_all = t < 0.0f;
    t2 = __fmul_rn(t, t);
  }
  int count = 0;
  float pen = 0.0f;
  for (int q = threadIdx.x; q < (J.cols >> 3); q += blockDim.x) {
    float acc[8];
    sumsq8(J.W + static_cast<size_t>(b) * B.block * J.ldw + (q << 3), B.block, J.ldw, acc);
    const size_t g0 = static_cast<size_t>(b) * J.cols + (q << 3);
    if (want_flags) {
      uint32_t lo = 0, hi = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t k0 = (keep_all || acc[i] > t2) ? 1u : 0u;
        const uint32_t k1 = (keep_all || acc[4 + i] > t2) ? 1u : 0u;
        lo |= k0 << (8 * i);
        hi |= k1 << (8 * i);
        count += static_cast<int>(k0 + k1);
      }
      *reinterpret_cast<uint2*>(J.flags + g0) = make_uint2(lo, hi);
    }
    if (want_norms) {
      float n[8], base[8], fresh[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        n[i] = norm_from_sumsq(acc[i]);
        base[i] = B.squared ? acc[i] : n[i];
        fresh[i] = reciprocal(base[i] + B.eps);
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
  // block totals: count (int) and penalty (float per thread, float64 from here on, fixed order)
  count = warp_sum(count);
  double pd = warp_sum(static_cast<double>(pen));
  const int warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  if ((threadIdx.x & 31) == 0) { s_cnt[warp] = count; s_pen[warp] = pd; }
  __syncthreads();
  if (threadIdx.x == 0) {
    int c = 0;
    double p = 0.0;
    for (int w = 0; w < n_warps; ++w) { c += s_cnt[w]; p += s_pen[w]; }
    if (want_flags) J.counts[b] = c;
    if (want_pen) {
      if (J.partial) J.partial[b] = p;
      else if (p != 0.0) atomicAdd(J.penalty, p);
    }
  }
}

// Rows staged in shared memory at a time: about 24 KB (the whole block for narrow matrices).
// With the 4-byte index list per column the dynamic shared memory stays under 48 KB for
// every width up to kFusedMaxCols.
__host__ __device__ inline int rows_per_pass(int cols) {
  int r = 12288 / cols;
  r = r < 3 ? 3 : r;
  return r > 16 ? 16 : r;
}
static_assert(kFusedMaxCols * (3 * 2 + 4) + 1024 <= 48 * 1024, "stage-2 shared memory must fit the default limit");

// Rows of a row-block that one stage-2 CTA handles: about 16K weights per CTA, a multiple of the
// 4-row staging pass, so that narrow matrices build their index list once per block and wide ones
// still spread over several CTAs.
__host__ __device__ inline int rows_per_cta(int cols, int d) {
  int r = (16384 / cols) / kRowsPerPass * kRowsPerPass;
  if (r < kRowsPerPass) r = kRowsPerPass;
  return r > d ? d : r;
}

__global__ void __launch_bounds__(256)
fused_stage2_kernel(const __grid_constant__ Batch B) {
  extern __shared__ __align__(16) uint8_t s_raw[];
  __shared__ int s_warp[32];
  __shared__ double s_red[8];
  __shared__ int s_base;
  const int j = find_job(B, blockIdx.x);
  const FusedJob& J = B.job[j];
  const int b = blockIdx.x - B.first_block[j];
  const int d = B.block;
  const int per_cta = rows_per_cta(J.cols, d);
  const int r_begin = blockIdx.y * per_cta;
  if (r_begin >= d) return;
  const int r_end = min(d, r_begin + per_cta);
  uint16_t* s_w = reinterpret_cast<uint16_t*>(s_raw);                                    // [rows_per_pass][cols]
  int32_t* s_idx = reinterpret_cast<int32_t*>(s_raw + static_cast<size_t>(rows_per_pass(J.cols)) * J.cols * 2);  // [cols]

  // penalty total of the job: its first CTA adds the per-block partials in a fixed order
  if (b == 0 && blockIdx.y == 0 && J.penalty != nullptr && J.partial != nullptr) {
    double p = 0.0;
    for (int i = threadIdx.x; i < J.n_blocks; i += blockDim.x) p += J.partial[i];
    p = warp_sum(p);
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = p;
    __syncthreads();
    if (threadIdx.x == 0) {
      double tot = 0.0;
      for (int w = 0; w < (blockDim.x >> 5); ++w) tot += s_red[w];
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

  const uint16_t* wblk = J.W + static_cast<size_t>(b) * d * J.ldw;
  const uint8_t* flags = J.flags + static_cast<size_t>(b) * J.cols;
  const int chunks = J.cols >> 3;

  // ascending list of kept columns: each thread inspects 8 flags per round
  if (kc > 0) {
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
  }
  if (kc == 0 && J.plan == nullptr) return;

  const bool vec_ok = (reinterpret_cast<uintptr_t>(J.vals) & 15) == 0;
  const long long tile0 = static_cast<long long>(d) * base;      // element offset of the block's tile in vals
  const int pass_rows = rows_per_pass(J.cols);
  for (int r_lo = r_begin; r_lo < r_end; r_lo += pass_rows) {
    const int n_rows = min(pass_rows, r_end - r_lo);
    // this pass's rows, one warp per row (rows warp, warp + n_warps, ...), lanes along the row:
    // 16-byte loads kept in shared memory; the execution layout is the same data with the pruned
    // columns zeroed.  No index arithmetic beyond adds, so the loop stays load-bound.
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
    for (int rr = warp; rr < n_rows; rr += n_warps) {
      const uint16_t* src = wblk + static_cast<size_t>(r_lo + rr) * J.ldw;
      uint16_t* dst = s_w + rr * J.cols;
      // (a plan that IS W: in-place mode, only pieces that change are written)
      const bool in_place = J.plan == J.W;
      uint16_t* pdst = J.plan ? J.plan + (static_cast<size_t>(b) * d + r_lo + rr) * (in_place ? J.ldw : J.cols) : nullptr;
      for (int q0 = lane; q0 < chunks; q0 += 128) {
        uint4 w[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (q0 + 32 * u < chunks) w[u] = __ldg(reinterpret_cast<const uint4*>(src + ((q0 + 32 * u) << 3)));
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int q = q0 + 32 * u;
          if (q >= chunks) break;
          *reinterpret_cast<uint4*>(dst + (q << 3)) = w[u];
          if (pdst != nullptr) {
            const uint2 f = *reinterpret_cast<const uint2*>(flags + (q << 3));
            uint4 m;   // a flag byte is 0 or 1: flag * 0xffff masks the matching 16-bit element
            m.x = w[u].x & (((f.x & 0xffu) * 0xffffu) | (((f.x >> 8) & 0xffu) * 0xffff0000u));
            m.y = w[u].y & ((((f.x >> 16) & 0xffu) * 0xffffu) | (((f.x >> 24) & 0xffu) * 0xffff0000u));
            m.z = w[u].z & (((f.y & 0xffu) * 0xffffu) | (((f.y >> 8) & 0xffu) * 0xffff0000u));
            m.w = w[u].w & ((((f.y >> 16) & 0xffu) * 0xffffu) | (((f.y >> 24) & 0xffu) * 0xffff0000u));
            if (!in_place || ((m.x ^ w[u].x) | (m.y ^ w[u].y) | (m.z ^ w[u].z) | (m.w ^ w[u].w)) != 0u)
              *reinterpret_cast<uint4*>(pdst + (q << 3)) = m;
          }
        }
      }
    }
    __syncthreads();   // s_w (and, on the first pass, s_idx) complete
    // packed tile rows of this pass, again one warp per row: row r occupies
    // vals[tile0 + r*kc, tile0 + (r+1)*kc); whole 16-byte vectors in the middle, ragged ends by element
    if (kc > 0) {
      for (int rr = warp; rr < n_rows; rr += n_warps) {
        const uint16_t* srow = s_w + rr * J.cols;
        const long long e0 = tile0 + static_cast<long long>(r_lo + rr) * kc;
        uint16_t* out_row = J.vals + e0;                               // element p of the row goes to out_row[p]
        if (vec_ok) {
          const int head = static_cast<int>((8 - (e0 & 7)) & 7);       // elements before the first aligned vector
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
    __syncthreads();   // s_w is overwritten by the next pass
  }
}

template <typename Fill>
int run_batches(const FusedJob* jobs, int n_jobs, int block, Fill launch) {
  for (int j0 = 0; j0 < n_jobs; j0 += kFusedMaxJobs) {
    Batch B;
    B.n_jobs = n_jobs - j0 < kFusedMaxJobs ? n_jobs - j0 : kFusedMaxJobs;
    B.block = block;
    int total = 0, max_cols = 0;
    for (int i = 0; i < B.n_jobs; ++i) {
      B.job[i] = jobs[j0 + i];
      B.first_block[i] = total;
      total += jobs[j0 + i].n_blocks;
      if (jobs[j0 + i].cols > max_cols) max_cols = jobs[j0 + i].cols;
    }
    B.first_block[B.n_jobs] = total;
    int st = launch(B, total, max_cols);
    if (st != BSP_OK) return st;
  }
  return BSP_OK;
}

}  // namespace

int fused_stage1(const FusedJob* jobs, int n_jobs, int block, float eps, int squared, cudaStream_t s) {
  return run_batches(jobs, n_jobs, block, [&](Batch& B, int total, int max_cols) -> int {
    B.eps = eps;
    B.squared = squared;
    int threads = ((max_cols >> 3) + 31) / 32 * 32;
    threads = threads > 256 ? 256 : threads;
    fused_stage1_kernel<<<total, threads, 0, s>>>(B);
    BSP_LAUNCH_CHECK();
    return BSP_OK;
  });
}

int fused_stage2(const FusedJob* jobs, int n_jobs, int block, cudaStream_t s) {
  return run_batches(jobs, n_jobs, block, [&](Batch& B, int total, int max_cols) -> int {
    B.eps = 0.0f;
    B.squared = 0;
    int splits = 1;
    for (int i = 0; i < B.n_jobs; ++i) {
      const int per = rows_per_cta(B.job[i].cols, block);
      const int need = (block + per - 1) / per;
      if (need > splits) splits = need;
    }
    size_t smem = 0;
    for (int i = 0; i < B.n_jobs; ++i) {
      const size_t need = static_cast<size_t>(B.job[i].cols) * (rows_per_pass(B.job[i].cols) * 2 + 4);
      if (need > smem) smem = need;
    }
    fused_stage2_kernel<<<dim3(total, splits), 256, smem, s>>>(B);
    BSP_LAUNCH_CHECK();
    return BSP_OK;
  });
}

}  // namespace bsp

extern "C" int bsp_prepare_batched(const bsp_layer_job* jobs, int n_jobs, int block, float eps, int pen,
                                   void* stream) {
  using namespace bsp;
  if (jobs == nullptr || n_jobs <= 0 || block <= 0) return BSP_ERR_ARG;
  if (pen != BSP_PEN_L2 && pen != BSP_PEN_L2SQ) return BSP_ERR_ARG;
  if (!(eps >= 0.0f)) return BSP_ERR_ARG;
  if (n_jobs > 4096) return BSP_ERR_UNSUPPORTED;
  // validate everything before the first launch
  for (int i = 0; i < n_jobs; ++i) {
    const bsp_layer_job& u = jobs[i];
    int st = check_matrix_args(u.W, u.rows, u.cols, u.ldw, block, BSP_ORIENT_C);
    if (st != BSP_OK) return st;
    if (u.blk_ptr == nullptr || u.idx == nullptr || u.vals == nullptr || u.ws == nullptr) return BSP_ERR_ARG;
    if (!aligned_to(u.ws, 256) || !aligned_to(u.blk_ptr, 4) || !aligned_to(u.idx, 4) || !aligned_to(u.vals, 2)) return BSP_ERR_ARG;
    if (u.threshold != u.threshold) return BSP_ERR_ARG;
    if (u.ws_bytes < ws_layout(u.rows / block, u.cols).total) return BSP_ERR_WORKSPACE;
    if (u.plan != nullptr && u.plan != u.W) {          // plan == W: in-place mode, W itself becomes the layout
      if (!aligned_to(u.plan, 256)) return BSP_ERR_ARG;
      if (u.plan_bytes < static_cast<size_t>(u.rows) * u.cols * 2) return BSP_ERR_WORKSPACE;
    }
    const bool ok = fused_shape_ok(u.W, u.rows, u.cols, u.ldw, block) && (u.keep == nullptr || aligned_to(u.keep, 8)) &&
                    (u.norms == nullptr || aligned_to(u.norms, 16)) && (u.gamma_out == nullptr || aligned_to(u.gamma_out, 16)) &&
                    (u.gamma_in == nullptr || aligned_to(u.gamma_in, 16));
    if (!ok) return BSP_ERR_UNSUPPORTED;
  }
  FusedJob* fj = new (std::nothrow) FusedJob[n_jobs];
  if (fj == nullptr) return BSP_ERR_ARG;
  for (int i = 0; i < n_jobs; ++i) {
    const bsp_layer_job& u = jobs[i];
    const int nb = u.rows / block;
    const WsLayout L = ws_layout(nb, u.cols);
    char* wsb = static_cast<char*>(u.ws);
    fj[i] = FusedJob{static_cast<const uint16_t*>(u.W), u.rows, u.cols, u.ldw, nb, u.threshold, u.threshold_dev,
                     u.norms, u.gamma_in, u.gamma_out, u.penalty, reinterpret_cast<double*>(wsb + L.sumsq_off),
                     u.keep ? u.keep : reinterpret_cast<uint8_t*>(wsb + L.keep_off),
                     reinterpret_cast<int32_t*>(wsb + L.counts_off), u.blk_ptr, u.idx, static_cast<uint16_t*>(u.vals),
                     u.kept_weights, static_cast<uint16_t*>(u.plan)};
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // The streaming one-pass kernel (W read once) takes the batch when every matrix fits its limits.  Its
  // per-item counts and penalty partials live in the workspace's S region, which this call does not use otherwise.
  int st = BSP_OK;
  bool done = false;
  {
    int32_t** pcounts = new (std::nothrow) int32_t*[n_jobs];
    double** ppartial = new (std::nothrow) double*[n_jobs];
    bool fits = pcounts != nullptr && ppartial != nullptr;
    for (int i = 0; i < n_jobs && fits; ++i) {
      const bsp_layer_job& u = jobs[i];
      const int nb = u.rows / block;
      const WsLayout L = ws_layout(nb, u.cols);
      char* region = static_cast<char*>(u.ws) + L.sumsq_off;          // 4 bytes per group
      const size_t slots = static_cast<size_t>(nb) * 32;              // at most 31 parts per block, plus two counters
      pcounts[i] = reinterpret_cast<int32_t*>(region);
      ppartial[i] = reinterpret_cast<double*>(region + round_up(slots * sizeof(int32_t), 256));
      if (round_up(slots * 4, 256) + slots * 8 > static_cast<size_t>(nb) * u.cols * 4) fits = false;
    }
    const int squared = pen == BSP_PEN_L2SQ ? 1 : 0;
    if (fits) st = fused_stream(fj, n_jobs, block, eps, squared, pcounts, ppartial, s, &done);
    delete[] pcounts;
    delete[] ppartial;
  }
  if (st == BSP_OK && !done) {
    st = fused_stage1(fj, n_jobs, block, eps, pen == BSP_PEN_L2SQ ? 1 : 0, s);
    if (st == BSP_OK) st = fused_stage2(fj, n_jobs, block, s);
  }
  delete[] fj;
  return st;
}
