// Streaming one-pass form of the vectorised weight-side kernels, for batches of any size: W is
// read from HBM exactly once.
//
// A work item is one row-block of one matrix (or a column range of it, so that its rows fit 24 KB
// of shared memory).  Items are numbered round by round across the matrices of the batch (see
// locate).  A CTA takes items from a ticket counter, so every item with a smaller number has been
// taken, and is being worked on, before; for each item it
//   load     has the item's rows brought into shared memory by bulk asynchronous copies (one per
//            row, all in flight at once, completion on an mbarrier);
//   phase A  computes the float32 sums of squares from shared memory (rows in increasing order, the
//            defined decision quantity), writes norms / gamma / keep flags, and publishes its kept
//            count (with a "ready" bit) and its penalty partial;
//   local    lists its kept columns and writes its part of the zero-expanded execution layout,
//            neither of which depends on other items;
//   phase B  reads the published counts of the items before it in the same matrix (bounded
//            relaxed loads), which give blk_ptr and the position of its part of the packed tile,
//            and writes indices and tile from shared memory.
// Shared memory per CTA is small (27 KB at 16-row blocks), so eight CTAs share an SM and their
// phases overlap: the latency of one item's chain is hidden by the other seven.
// Why this cannot deadlock: a published count depends on nobody, and a taken item is published
// without waiting.  An item waits for items with a smaller number (all taken) and, when its
// row-block is split into column ranges, for the later ranges of its own block, which are the next
// tickets; at most one block straddles the ticket counter, so fewer than 32 CTAs can wait for items
// nobody has taken, and the GPU holds more CTAs than that at once.  A CTA takes its next ticket only
// after the last wait of its current item, so a ticket is never held by a CTA that is waiting.
// A batch of at most one wave of CTAs runs without the counter (item = block index): it relies on
// the hardware starting the blocks of a grid in index order, as it does; were that ever not so, the
// bounded waits would end the launch with BSP_ERR_TIMEOUT rather than hang it.
// Counts and penalty partials are published as single words that carry their own "ready" bit (the
// lowest mantissa bit of the float64 partial), read with relaxed loads: a reader needs nothing but
// the word itself, so no fence is involved.  The last item of a matrix adds the partials in a fixed
// order.  Masks, indices, tiles, norms and gamma are bit-identical to the two-stage path.
#include <cstddef>
#include <cstring>
#include <new>

#include "bsp_tc.cuh"

namespace bsp {
namespace {

using tc::mbar_init;
using tc::mbar_arrive_expect_tx;
using tc::mbar_wait;
using tc::smem_u32;

constexpr int kStreamMaxJobs = 96;       // per launch; the job table travels as a kernel parameter
constexpr int kStreamThreads = 128;
constexpr int kStreamRowBytes = 24 * 1024;   // the row buffer
constexpr int kReadyBit = 0x40000000;    // set in a published count

struct StreamJob {
  FusedJob j;
  int parts, part_cols;      // column ranges per row-block, columns per range (multiple of 8)
  int seg_round;             // first round of this matrix's segment (see locate) = row-blocks of the previous matrix
  int32_t* part_counts;      // [n_blocks * parts] published counts, then (job 0) the ticket
  unsigned long long* part_partial;   // [n_blocks * parts] published penalty partials (float64 bits, lowest bit set)
};
template <int N>
struct StreamBatchT {
  int n_jobs, block, squared;
  float eps;
  int total_items, buf_bytes;
  int parts_total;           // column ranges of one round over every matrix of the batch
  int sms, stagger_ns;       // start of the CTAs that share an SM, one after the other (ticket variant)
  int* ticket;
  int* status;               // receives BSP_ERR_TIMEOUT when a bounded wait expires
  // Item order (see locate): the table is sorted by row-block count; a matrix's "segment" is the run of
  // rounds in which it is the smallest matrix still active.  The two arrays that locate searches are kept
  // apart from the wide job records, so that a search stays within a few lines of the constant cache.
  int seg_item[N];           // number of the first item of the matrix's segment
  int parts_before[N];       // column ranges per round of the matrices before this one in the table
  StreamJob job[N];
};
// The job table travels as a kernel parameter: 14 KB for a full batch, which every launch has to
// move; a batch of up to eight matrices (an encoder layer's) gets a table of 1.2 KB with the same fields.
constexpr int kStreamFewJobs = 8;
using StreamBatch = StreamBatchT<kStreamMaxJobs>;

struct Item {
  int jn, local, b, q, c0, pc;
};
// Items are numbered round by round: round r holds row-block r of every matrix that has one, matrix
// after matrix, the column ranges of a block side by side.  The row-blocks of one matrix are therefore
// a whole round apart, so the items whose counts an item needs were taken long before it (all but the
// last few have finished), while a matrix-after-matrix order would make every item wait for the
// slowest of some hundred items that started together with it.
template <class Batch>
__device__ __forceinline__ Item locate(const Batch& B, int item) {
  int lo = 0, hi = B.n_jobs - 1;
  while (lo < hi) {                    // the segment: the last matrix whose segment starts at or before the item
    const int mid = (lo + hi + 1) >> 1;
    if (B.seg_item[mid] <= item) lo = mid; else hi = mid - 1;
  }
  const int seg_round = B.job[lo].seg_round;
  const int per_round = B.parts_total - B.parts_before[lo];
  const int u = item - B.seg_item[lo];
  const int round = u / per_round;
  const int o = u - round * per_round + B.parts_before[lo];
  hi = B.n_jobs - 1;
  while (lo < hi) {                    // the matrix: the last one whose ranges start at or before o
    const int mid = (lo + hi + 1) >> 1;
    if (B.parts_before[mid] <= o) lo = mid; else hi = mid - 1;
  }
  const StreamJob& O = B.job[lo];
  Item I;
  I.jn = lo;
  I.b = seg_round + round;
  I.q = o - B.parts_before[lo];
  I.local = I.b * O.parts + I.q;
  I.c0 = I.q * O.part_cols;
  I.pc = min(O.part_cols, O.j.cols - I.c0);
  return I;
}

// Rows of an item into a shared-memory buffer, one bulk copy per row (called by one warp).
template <class Batch>
__device__ __forceinline__ void issue_rows(const Batch& B, const Item& I, uint32_t dst, uint32_t bar, int lane) {
  const FusedJob& J = B.job[I.jn].j;
  const int d = B.block;
  const uint32_t row_bytes = static_cast<uint32_t>(I.pc) * 2u;
  if (lane == 0) mbar_arrive_expect_tx(bar, row_bytes * static_cast<uint32_t>(d));
  __syncwarp();
  const uint16_t* wblk = J.W + static_cast<size_t>(I.b) * d * J.ldw + I.c0;
  for (int r = lane; r < d; r += 32) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst + static_cast<uint32_t>(r) * row_bytes),
                   "l"(reinterpret_cast<uint64_t>(wblk + static_cast<size_t>(r) * J.ldw)), "r"(row_bytes), "r"(bar)
                 : "memory");
  }
}

// Published word of an item as it is now (ready bit set or not).
__device__ __forceinline__ int probe_count(const int32_t* slot) {
  int v;
  asm volatile("ld.relaxed.gpu.global.b32 %0, [%1];" : "=r"(v) : "l"(slot) : "memory");
  return v;
}
// Published count of an item: waits (bounded) for its ready bit.  The limit is fetched only after
// the first round of probes, so the usual short wait costs no extra trip to memory.
__device__ __forceinline__ int wait_count(const int32_t* slot, int* status) {
  unsigned long long limit = 0, start = 0;
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) {
      const int v = probe_count(slot);
      if (v & kReadyBit) return v & (kReadyBit - 1);
      __nanosleep(32);
    }
    if (limit == 0) {
      limit = tc::wait_limit_ns(status);
      start = tc::global_timer_ns();
    } else if (tc::global_timer_ns() - start > limit) {
      atomicExch(status, BSP_ERR_TIMEOUT);
      return 0;
    }
  }
}

// Up to four published counts, words slot[0], slot[stride], ...: v[u] holds what an earlier probe saw
// (any word with the ready bit is final).  Words that are not ready are asked for again, all of them
// at once, until every one is; returns the sum of the counts.  n = how many of the four exist.
__device__ __forceinline__ int wait_counts4(const int32_t* slot, int stride, int n, int (&v)[4], int* status) {
  unsigned long long limit = 0, start = 0;
  for (int round = 0;; ++round) {
    bool all = true;
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (u < n && !(v[u] & kReadyBit)) v[u] = probe_count(slot + u * stride);
#pragma unroll
    for (int u = 0; u < 4; ++u) all = all && (u >= n || (v[u] & kReadyBit) != 0);
    if (all) break;
    __nanosleep(32);
    if ((round & 63) == 63) {
      if (limit == 0) {
        limit = tc::wait_limit_ns(status);
        start = tc::global_timer_ns();
      } else if (tc::global_timer_ns() - start > limit) {
        atomicExch(status, BSP_ERR_TIMEOUT);
        return 0;
      }
    }
  }
  int sum = 0;
#pragma unroll
  for (int u = 0; u < 4; ++u) sum += u < n ? (v[u] & (kReadyBit - 1)) : 0;
  return sum;
}

// Published penalty partial of an item: waits (bounded) for its ready bit.
__device__ __forceinline__ double wait_partial(const unsigned long long* slot, int* status) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.b64 %0, [%1];" : "=l"(v) : "l"(slot) : "memory");
  if (v & 1ull) return __longlong_as_double(static_cast<long long>(v));
  const unsigned long long limit = tc::wait_limit_ns(status);
  const unsigned long long start = tc::global_timer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) {
      asm volatile("ld.relaxed.gpu.global.b64 %0, [%1];" : "=l"(v) : "l"(slot) : "memory");
      if (v & 1ull) return __longlong_as_double(static_cast<long long>(v));
      __nanosleep(32);
    }
    if (tc::global_timer_ns() - start > limit) { atomicExch(status, BSP_ERR_TIMEOUT); return 0.0; }
  }
}

// kOneWave: the batch fits the GPU in one wave (every CTA resident, item = block index, no ticket).
// All items then start together and every one of them waits for the slowest of the items before it,
// so the packed tile is built in shared memory while that wait lasts; with tickets the counts an item
// needs are ready long before it asks, and the tile goes from the row buffer straight to memory.
template <int N, bool kOneWave>
__global__ void __launch_bounds__(kStreamThreads, 8)
fused_stream_kernel(const __grid_constant__ StreamBatchT<N> B) {
  extern __shared__ __align__(128) uint8_t s_raw[];
  __shared__ __align__(8) uint64_t s_bar;
  __shared__ int s_item;
  __shared__ int s_cnt[8];
  __shared__ double s_pen[8];
  __shared__ int s_warp[32];
  __shared__ int s_sum[3];
  __shared__ int s_kc;
  const int d = B.block;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
  uint16_t* s_idx = reinterpret_cast<uint16_t*>(s_raw + static_cast<size_t>(B.buf_bytes));    // [max part columns], local column numbers
  const uint32_t bar = smem_u32(&s_bar);

  // A batch that fits the GPU in one wave needs no ticket: every CTA is resident, item = block index,
  // and the item's job is looked up (which brings its part of the kernel parameters into the constant
  // cache) while the clearing kernel is still running.
  constexpr bool direct = kOneWave;
  int item = static_cast<int>(blockIdx.x);
  Item I = locate(B, direct ? item : 0);
  if (direct) {
    const FusedJob& J0 = B.job[I.jn].j;
    asm volatile("" ::"l"(J0.W), "r"(J0.ldw), "l"(J0.flags), "l"(J0.vals), "l"(B.job[I.jn].part_counts));
  }
  if (warp == 0) {
    if (lane == 0) {
      mbar_init(bar, 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    // One wave: the rows are asked for before the wait for the clearing kernel.  That kernel is an
    // ordinary launch, so whatever wrote W earlier in the stream had finished before it began, and
    // this grid was started after that; only the published counts depend on the clearing itself.
    if (direct) issue_rows(B, I, smem_u32(s_raw), bar, lane);
  }
  if (threadIdx.x == 0) {
    // launched with programmatic stream serialization: everything above overlapped the clearing
    // kernel; the ticket and the slots it zeroes are touched only from here on
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may set up on SMs that become free
    if (!direct) {
      // CTAs that start together and work on items of one size stay in step: all of an SM's CTAs load,
      // then all compute.  The k-th CTA of an SM (block numbers go round the SMs) therefore takes its
      // first ticket k * stagger later, so that loads and arithmetic of different CTAs overlap.
      const unsigned long long delay = static_cast<unsigned long long>(blockIdx.x / B.sms) * B.stagger_ns;
      if (delay) {
        const unsigned long long t0 = tc::global_timer_ns();
        while (tc::global_timer_ns() - t0 < delay) __nanosleep(100);
      }
      s_item = atomicAdd(B.ticket, 1);
    }
  }
  __syncthreads();
  if (!direct) {
    item = s_item;
    if (item >= B.total_items) return;
    I = locate(B, item);
  }
  // A CTA works through items until the tickets run out.  It takes its next ticket only when every
  // wait of the current item is behind it (what is left then, writing indices and the tile, waits for
  // nobody), so an item is never held by a CTA that is itself waiting, and the trip to the ticket
  // counter overlaps those writes.
  uint32_t parity = 0u;
  for (;;) {
    if (warp == 0 && !direct) issue_rows(B, I, smem_u32(s_raw), bar, lane);
    const StreamJob& O = B.job[I.jn];
    const FusedJob& J = O.j;
    const int b = I.b, q = I.q, c0 = I.c0, pc = I.pc, local = I.local;
    const int chunks = pc >> 3;
    const uint16_t* s_w = reinterpret_cast<const uint16_t*>(s_raw);                     // [d][pc]
    uint8_t* s_flag = reinterpret_cast<uint8_t*>(s_idx + O.part_cols);                  // [pc]
    // one decision for the whole CTA; if the rows never arrived, hold the buffer a millisecond for
    // copies that may still be on their way, then leave
    if (!__syncthreads_and(tc::mbar_wait_suspended(bar, parity, B.status) ? 1 : 0)) {
      if (threadIdx.x == 0) atomicExch(B.status, BSP_ERR_TIMEOUT);
      const unsigned long long start = tc::global_timer_ns();
      while (tc::global_timer_ns() - start < tc::kQuietNs) __nanosleep(2000);
      return;
    }

    // ---- phase A: sums of squares of 8 adjacent columns per thread, rows in increasing order
    const bool want_pen = J.penalty != nullptr;
    const bool want_norms = J.norms != nullptr || J.gamma_out != nullptr || want_pen;
    const float t = J.threshold_dev ? *J.threshold_dev : J.threshold;
    const bool keep_all = t < 0.0f;
    const float t2 = __fmul_rn(t, t);
    int count = 0;
    float pen = 0.0f;
    const bool in_place = J.plan != nullptr && J.plan == J.W;
    int changes = 0;                         // in-place mode: a pruned group that still holds a non-zero weight
    for (int k = threadIdx.x; k < chunks; k += blockDim.x) {
      float acc[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] = 0.0f;
#pragma unroll 4
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
        changes |= static_cast<int>((k0 == 0u && acc[i] != 0.0f) || (k1 == 0u && acc[4 + i] != 0.0f));
      }
      const size_t g0 = static_cast<size_t>(b) * J.cols + c0 + (k << 3);
      *reinterpret_cast<uint2*>(s_flag + (k << 3)) = make_uint2(lo, hi);
      *reinterpret_cast<uint2*>(J.flags + g0) = make_uint2(lo, hi);
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
    count = warp_sum(count);
    double pd = warp_sum(static_cast<double>(pen));
    if (lane == 0) { s_cnt[warp] = count; s_pen[warp] = pd; }
    const bool rewrite = __syncthreads_or(changes) != 0;     // (the block-wide barrier of this point)
    const int n_parts = J.n_blocks * O.parts;
    if (threadIdx.x == 0) {
      int c = 0;
      double p = 0.0;
      for (int w = 0; w < n_warps; ++w) { c += s_cnt[w]; p += s_pen[w]; }
      asm volatile("st.relaxed.gpu.global.b32 [%0], %1;" ::"l"(O.part_counts + local), "r"(c | kReadyBit) : "memory");
      if (want_pen)
        asm volatile("st.relaxed.gpu.global.b64 [%0], %1;" ::"l"(O.part_partial + local),
                     "l"(static_cast<unsigned long long>(__double_as_longlong(p)) | 1ull) : "memory");
      s_kc = c;
      s_sum[0] = 0; s_sum[1] = 0; s_sum[2] = 0;
    }

    // ---- local work: ascending list of this part's kept columns (local indices in s_idx)
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
        if (bit) s_idx[p++] = static_cast<uint16_t>((k << 3) + i);
      }
    }
    // execution layout: the rows with the pruned columns zeroed, one warp per row, 16-byte stores.
    // When the job's plan IS its W (in-place mode, Algorithm 2's W = W * Mask), only 8-column pieces
    // that hold a weight of a pruned group are written: W read once, and written only where it changes
    // (an item whose pruned groups are all zero already skips the pass).
    if (J.plan != nullptr && (!in_place || rewrite)) {
      const size_t pld = in_place ? static_cast<size_t>(J.ldw) : static_cast<size_t>(J.cols);
      for (int r = warp; r < d; r += n_warps) {
        uint16_t* pdst = J.plan + (static_cast<size_t>(b) * d + r) * pld + c0;
        for (int k = lane; k < chunks; k += 32) {
          const uint4 w = *reinterpret_cast<const uint4*>(s_w + r * pc + (k << 3));
          const uint2 f = *reinterpret_cast<const uint2*>(s_flag + (k << 3));
          uint4 m;   // a flag byte is 0 or 1: flag * 0xffff masks the matching 16-bit element
          m.x = w.x & (((f.x & 0xffu) * 0xffffu) | (((f.x >> 8) & 0xffu) * 0xffff0000u));
          m.y = w.y & ((((f.x >> 16) & 0xffu) * 0xffffu) | (((f.x >> 24) & 0xffu) * 0xffff0000u));
          m.z = w.z & (((f.y & 0xffu) * 0xffffu) | (((f.y >> 8) & 0xffu) * 0xffff0000u));
          m.w = w.w & ((((f.y >> 16) & 0xffu) * 0xffffu) | (((f.y >> 24) & 0xffu) * 0xffff0000u));
          if (!in_place || ((m.x ^ w.x) | (m.y ^ w.y) | (m.z ^ w.z) | (m.w ^ w.w)) != 0u)
            *reinterpret_cast<uint4*>(pdst + (k << 3)) = m;
        }
      }
    }

    if constexpr (kOneWave) {
    // ---- local work, continued: the packed tile of this part, built in place.  Row r's kept values
    // move to the front of row r in the row buffer (position p comes from column idx[p] >= p, so moving
    // left in ascending order never overwrites a value that is still needed).  Nothing here depends on
    // other items: the trip of the published counts through memory (phase B) overlaps it, and what is
    // left once the offsets are known is a copy of contiguous rows.
    // A lane takes two neighbouring kept positions: their column numbers are one 32-bit word of the
    // list and the two values lie about six columns apart (three banks from lane to lane at the usual
    // densities, where eight positions per lane would put four lanes on each bank).  A warp owns its
    // rows from here to the end of the item; it handles 32 pairs of four rows at a time: reads, then
    // writes, with the reads of later pairs lying beyond everything written so far.
    __syncthreads();                          // the list is complete and the execution-layout pass has read the rows
    {
      const int kc_part = s_kc;
      const int n_pairs = kc_part >> 1;
      uint16_t* s_wm = reinterpret_cast<uint16_t*>(s_raw);
      uint32_t* s_w32 = reinterpret_cast<uint32_t*>(s_raw);
      const int row_words = pc >> 1;
      for (int c = 0; c < n_pairs; c += 32) {
        const int pp = c + lane;
        const bool on = pp < n_pairs;
        const uint32_t cc = on ? *reinterpret_cast<const uint32_t*>(s_idx + 2 * pp) : 0u;
        const uint16_t* sa = s_wm + (cc & 0xffffu);
        const uint16_t* sb = s_wm + (cc >> 16);
        for (int r = warp; r < d; r += 4 * n_warps) {
          uint32_t w[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int rr = r + u * n_warps;
            if (on && rr < d) w[u] = static_cast<uint32_t>(sa[rr * pc]) | (static_cast<uint32_t>(sb[rr * pc]) << 16);
          }
          __syncwarp();
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int rr = r + u * n_warps;
            if (on && rr < d) s_w32[rr * row_words + pp] = w[u];
          }
        }
        __syncwarp();
      }
      if (kc_part & 1) {                      // an odd count: the last position, after every pair (its source lies beyond them)
        const int p = kc_part - 1;
        const int col = s_idx[p];
        for (int r = warp + lane * n_warps; r < d; r += 32 * n_warps) s_wm[r * pc + p] = s_wm[r * pc + col];
      }
    }
    }

    // ---- phase B: offsets from the published counts
    // (a thread asks for all its words before it waits for any: the trips to memory overlap.  Asking
    // earlier, before the local work, made the waits longer, not shorter: measured.)
    int before = 0, in_block_before = 0, in_block = 0;
    const int mine_part = static_cast<int>(threadIdx.x) < O.parts && O.parts > 1 ? static_cast<int>(threadIdx.x) : -1;   // parts <= 31
    int pv = mine_part >= 0 ? probe_count(O.part_counts + b * O.parts + mine_part) : 0;
    for (int i0 = threadIdx.x; i0 < local; i0 += 4 * blockDim.x) {
      int v[4] = {0, 0, 0, 0};
      const int n = (local - i0 + static_cast<int>(blockDim.x) - 1) / static_cast<int>(blockDim.x);   // words of this thread in this round (capped at four below)
      before += wait_counts4(O.part_counts + i0, static_cast<int>(blockDim.x), n < 4 ? n : 4, v, B.status);
    }
    if (mine_part >= 0) {
      if (!(pv & kReadyBit)) pv = wait_count(O.part_counts + b * O.parts + mine_part, B.status);
      pv &= kReadyBit - 1;
      in_block = pv;
      if (mine_part < q) in_block_before = pv;
    }
    before = warp_sum(before);
    in_block = warp_sum(in_block);
    in_block_before = warp_sum(in_block_before);
    __syncthreads();                          // s_sum zeroed, s_kc set, s_idx complete
    if (lane == 0) {
      if (before) atomicAdd(&s_sum[0], before);
      if (in_block) atomicAdd(&s_sum[1], in_block);
      if (in_block_before) atomicAdd(&s_sum[2], in_block_before);
    }
    __syncthreads();
    const int kc = s_kc;                     // kept groups of this part
    const int base = s_sum[0];               // kept groups before this item's first one (index into idx)
    const int kc_block = O.parts > 1 ? s_sum[1] : kc;   // kept groups of the whole row-block
    const int off_in_block = s_sum[2];       // kept groups of the block's earlier parts
    const int block_base = base - off_in_block;
    if (q == 0 && threadIdx.x == 0) {
      J.blk_ptr[b] = block_base;
      if (b == J.n_blocks - 1) {
        J.blk_ptr[J.n_blocks] = block_base + kc_block;
        if (J.kept_weights) *J.kept_weights = static_cast<int64_t>(block_base + kc_block) * d;
      }
    }
    // penalty total of the matrix, in a fixed order, by its last item (every other item has a smaller number)
    if (local == n_parts - 1 && want_pen) {
      double p = 0.0;
      for (int i = threadIdx.x; i < n_parts; i += blockDim.x) p += wait_partial(O.part_partial + i, B.status);
      p = warp_sum(p);
      if (lane == 0) s_pen[warp] = p;
      __syncthreads();
      if (threadIdx.x == 0) {
        double tot = 0.0;
        for (int w = 0; w < n_warps; ++w) tot += s_pen[w];
        *J.penalty = tot;
      }
    }
    // no wait from here on: take the next item (the answer is only looked at after the writes below)
    int next_item = 0;
    if (!direct && threadIdx.x == 0) next_item = atomicAdd(B.ticket, 1);
    if (kc > 0) {
      for (int p = threadIdx.x; p < kc; p += blockDim.x) J.idx[base + p] = c0 + s_idx[p];
      // packed tile: row r of the block occupies vals[tile0 + r*kc_block, +kc_block); this part fills
      // positions [off_in_block, off_in_block + kc) of every row.
      const long long tile0 = static_cast<long long>(d) * block_base;
      const uintptr_t vals_addr = reinterpret_cast<uintptr_t>(J.vals);
      if constexpr (kOneWave) {
        // from the front of row r of the buffer, where the values were gathered above.  Each warp copies
        // the rows it compacted: 16-byte pieces where the destination row is aligned (the source is),
        // 4-byte pieces or single elements otherwise.
        __syncwarp();
        for (int r = warp; r < d; r += n_warps) {
          const uint16_t* srow = s_w + r * pc;
          const long long e0 = tile0 + static_cast<long long>(r) * kc_block + off_in_block;
          uint16_t* out_row = J.vals + e0;
          int done = 0;
          if ((vals_addr & 15) == 0 && (e0 & 7) == 0) {
            const int n_vec = kc >> 3;
            for (int v = lane; v < n_vec; v += 32)
              *reinterpret_cast<uint4*>(out_row + (v << 3)) = *reinterpret_cast<const uint4*>(srow + (v << 3));
            done = n_vec << 3;
          } else if ((vals_addr & 3) == 0 && (e0 & 1) == 0) {
            const int n_w = kc >> 1;
            for (int v = lane; v < n_w; v += 32)
              *reinterpret_cast<uint32_t*>(out_row + (v << 1)) = *reinterpret_cast<const uint32_t*>(srow + (v << 1));
            done = n_w << 1;
          }
          for (int p = done + lane; p < kc; p += 32) out_row[p] = srow[p];
        }
      } else if ((vals_addr & 3) == 0 && ((kc_block | off_in_block) & 1) == 0 && (tile0 & 1) == 0) {
        // Every row of this part starts on a 4-byte boundary.  A lane takes two neighbouring kept
        // positions (one word of the list, two values about six columns apart: different banks from lane
        // to lane) and the pair leaves as one 4-byte store, 128 contiguous bytes per warp; four rows of
        // the warp at a time, eight loads in flight.
        const int n_pairs = kc >> 1;
        uint32_t* out32 = reinterpret_cast<uint32_t*>(J.vals + tile0 + off_in_block);
        const size_t row_words = static_cast<size_t>(kc_block >> 1);
        for (int pp = lane; pp < n_pairs; pp += 32) {
          const uint32_t cc = *reinterpret_cast<const uint32_t*>(s_idx + 2 * pp);
          const uint16_t* sa = s_w + (cc & 0xffffu);
          const uint16_t* sb = s_w + (cc >> 16);
          uint32_t* o = out32 + pp;
          for (int r = warp; r < d; r += 4 * n_warps) {
            uint32_t w[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int rr = r + u * n_warps;
              if (rr < d) w[u] = static_cast<uint32_t>(sa[rr * pc]) | (static_cast<uint32_t>(sb[rr * pc]) << 16);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int rr = r + u * n_warps;
              if (rr < d) o[static_cast<size_t>(rr) * row_words] = w[u];
            }
          }
        }
        if (kc & 1) {                         // an odd part of a split row-block: its last position, one thread per row
          const int p = kc - 1;
          for (int rr = threadIdx.x; rr < d; rr += blockDim.x)
            J.vals[tile0 + static_cast<long long>(rr) * kc_block + off_in_block + p] = s_w[rr * pc + s_idx[p]];
        }
      } else {
        for (int r = warp; r < d; r += n_warps) {
          const uint16_t* srow = s_w + r * pc;
          uint16_t* out_row = J.vals + tile0 + static_cast<long long>(r) * kc_block + off_in_block;
          for (int p = lane; p < kc; p += 32) out_row[p] = srow[s_idx[p]];
        }
      }
    }
    if (direct) break;
    if (threadIdx.x == 0) s_item = next_item;
    __syncthreads();                         // everybody is done with the row buffer and the lists; s_item is there
    item = s_item;
    if (item >= B.total_items) break;
    I = locate(B, item);
    parity ^= 1u;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the buffer's readers are done before the copies write it
  }
}

// Zeroes the published counts and partials and the ticket slot of every matrix.
template <int N>
__global__ void __launch_bounds__(256)
stream_clear_kernel(const __grid_constant__ StreamBatchT<N> B) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the main kernel may take its seats now; it waits for this grid
  const StreamJob& O = B.job[blockIdx.x];
  const int n = O.j.n_blocks * O.parts;
  for (int i = threadIdx.x; i < n + 2; i += blockDim.x) O.part_counts[i] = 0;
  for (int i = threadIdx.x; i < n; i += blockDim.x) O.part_partial[i] = 0ull;
}

int total_parts_so_far(const StreamBatch& B, int n) {
  int p = 0;
  for (int i = 0; i < n; ++i) p += B.job[i].parts;
  return p;
}

// Fills the job table; false when a matrix does not fit this kernel's limits.
bool fill_batch(StreamBatch& B, const FusedJob* jobs, int n_jobs, int block, float eps, int squared,
                int32_t* const* part_counts, double* const* part_partial, size_t* smem_out) {
  B.n_jobs = n_jobs;
  B.block = block;
  B.squared = squared;
  B.eps = eps;
  int total = 0, max_part_cols = 0;
  const int max_cols = (kStreamRowBytes / (2 * block)) / 8 * 8;        // columns whose rows fit a row buffer
  if (max_cols < 8) return false;
  // table order: ascending row-block count (insertion sort, stable; at most 96 entries)
  int order[kStreamMaxJobs];
  for (int i = 0; i < n_jobs; ++i) {
    int k = i;
    while (k > 0 && jobs[order[k - 1]].n_blocks > jobs[i].n_blocks) { order[k] = order[k - 1]; --k; }
    order[k] = i;
  }
  for (int i = 0; i < n_jobs; ++i) {
    StreamJob& O = B.job[i];
    const int src = order[i];
    O.j = jobs[src];
    const int cols = O.j.cols;
    O.parts = (cols + max_cols - 1) / max_cols;
    O.part_cols = ((cols + O.parts - 1) / O.parts + 7) / 8 * 8;
    O.parts = (cols + O.part_cols - 1) / O.part_cols;
    if (O.parts > 31) return false;
    if (static_cast<long long>(O.j.n_blocks) * O.parts + 2 > static_cast<long long>(O.j.n_blocks) * 32) return false;
    O.part_counts = part_counts[src];
    O.part_partial = reinterpret_cast<unsigned long long*>(part_partial[src]);
    B.parts_before[i] = total_parts_so_far(B, i);
    total += O.j.n_blocks * O.parts;
    if (O.part_cols > max_part_cols) max_part_cols = O.part_cols;
  }
  B.total_items = total;
  B.parts_total = total_parts_so_far(B, n_jobs);
  int seg_item = 0, prev_blocks = 0;
  for (int i = 0; i < n_jobs; ++i) {
    StreamJob& O = B.job[i];
    B.seg_item[i] = seg_item;
    O.seg_round = prev_blocks;
    seg_item += (O.j.n_blocks - prev_blocks) * (B.parts_total - B.parts_before[i]);
    prev_blocks = O.j.n_blocks;
  }
  B.buf_bytes = static_cast<int>(round_up(static_cast<size_t>(block) * max_part_cols * 2, 128));
  B.ticket = B.job[0].part_counts + B.job[0].j.n_blocks * B.job[0].parts + 1;
  *smem_out = static_cast<size_t>(B.buf_bytes) + static_cast<size_t>(max_part_cols) * 3 + 16;   // rows, 2-byte list, flags
  return true;
}

}  // namespace

// Runs the batch through the streaming one-pass kernel (a clearing launch and the kernel, per 96
// matrices).  *used = false means nothing was launched and the two-stage path should run.
int fused_stream(const FusedJob* jobs, int n_jobs, int block, float eps, int squared, int32_t* const* part_counts,
                 double* const* part_partial, cudaStream_t s, bool* used) {
  *used = false;
  TcDevice* td = tc_device();
  if (td == nullptr) return BSP_ERR_CUDA;
  StreamBatch* B = new (std::nothrow) StreamBatch;
  if (B == nullptr) return BSP_OK;
  // every batch is checked before the first launch
  size_t smem = 0, smem_max = 0;
  bool ok = true;
  for (int j0 = 0; j0 < n_jobs && ok; j0 += kStreamMaxJobs) {
    const int n = n_jobs - j0 < kStreamMaxJobs ? n_jobs - j0 : kStreamMaxJobs;
    ok = fill_batch(*B, jobs + j0, n, block, eps, squared, part_counts + j0, part_partial + j0, &smem);
    if (smem > smem_max) smem_max = smem;
  }
  constexpr int kSmemCap = 96 * 1024;     // opt-in limit set once per device; a launch asks for what it needs
  if (ok && smem_max > static_cast<size_t>(kSmemCap)) ok = false;
  int per_sm = 0;
  int st = BSP_OK;
  if (ok) {
    if (!td->attr_set[7]) {
      cudaError_t e = cudaFuncSetAttribute(fused_stream_kernel<kStreamMaxJobs, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemCap);
      if (e == cudaSuccess)
        e = cudaFuncSetAttribute(fused_stream_kernel<kStreamMaxJobs, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemCap);
      if (e == cudaSuccess)
        e = cudaFuncSetAttribute(fused_stream_kernel<kStreamFewJobs, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemCap);
      if (e == cudaSuccess)
        e = cudaFuncSetAttribute(fused_stream_kernel<kStreamFewJobs, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemCap);
      if (e != cudaSuccess) { delete B; return cuda_fail(e); }
      td->attr_set[7] = true;
    }
    int per_sm_one_wave = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fused_stream_kernel<kStreamMaxJobs, false>, kStreamThreads, smem_max);
    if (e == cudaSuccess)
      e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm_one_wave, fused_stream_kernel<kStreamMaxJobs, true>, kStreamThreads, smem_max);
    if (e != cudaSuccess) { delete B; return cuda_fail(e); }
    if (per_sm_one_wave < per_sm) per_sm = per_sm_one_wave;      // "one wave" must hold for the variant that assumes it
    if (per_sm * td->sms < 32) ok = false;    // the no-deadlock argument needs 32 CTAs resident at once
  }
  for (int j0 = 0; j0 < n_jobs && ok && st == BSP_OK; j0 += kStreamMaxJobs) {
    const int n = n_jobs - j0 < kStreamMaxJobs ? n_jobs - j0 : kStreamMaxJobs;
    fill_batch(*B, jobs + j0, n, block, eps, squared, part_counts + j0, part_partial + j0, &smem);
    B->status = td->status;
    B->sms = td->sms;
    // (measured on the 72-matrix stack: 80.8 us without, 76.8 / 74.8 / 76.8 / 78.8 us at 400 / 800 / 1200 / 1600 ns;
    // a batch of only a few waves would lose more at the start than it gains)
    B->stagger_ns = B->total_items >= 4 * per_sm * td->sms ? 750 : 0;
    if (B->total_items <= per_sm * td->sms) B->ticket = nullptr;    // one wave: item = block index
    const bool few = n <= kStreamFewJobs;
    StreamBatchT<kStreamFewJobs> small;
    if (few) {
      memcpy(&small, B, offsetof(StreamBatch, seg_item));      // the scalar fields come first in both
      for (int i = 0; i < kStreamFewJobs; ++i) {
        small.seg_item[i] = B->seg_item[i];
        small.parts_before[i] = B->parts_before[i];
        small.job[i] = B->job[i];
      }
      stream_clear_kernel<kStreamFewJobs><<<n, 256, 0, s>>>(small);
    } else {
      stream_clear_kernel<kStreamMaxJobs><<<n, 256, 0, s>>>(*B);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { st = cuda_fail(e); break; }
    cudaLaunchConfig_t cfg = {};
    const int resident = per_sm * td->sms;
    cfg.gridDim = dim3(B->total_items < resident ? B->total_items : resident);   // CTAs loop until the tickets run out
    cfg.blockDim = dim3(kStreamThreads);
    cfg.dynamicSmemBytes = smem_max;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // start while the clearing kernel drains
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const bool one_wave = B->ticket == nullptr;
    e = few ? (one_wave ? cudaLaunchKernelEx(&cfg, fused_stream_kernel<kStreamFewJobs, true>, small)
                        : cudaLaunchKernelEx(&cfg, fused_stream_kernel<kStreamFewJobs, false>, small))
            : (one_wave ? cudaLaunchKernelEx(&cfg, fused_stream_kernel<kStreamMaxJobs, true>, *B)
                        : cudaLaunchKernelEx(&cfg, fused_stream_kernel<kStreamMaxJobs, false>, *B));
    if (e != cudaSuccess) { st = cuda_fail(e); break; }
    *used = true;
  }
  delete B;
  return st;
}

}  // namespace bsp
