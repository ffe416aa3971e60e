// bsp_linear_gathered: the pruned linear layer with the pruned work skipped.  For a row-block of
// d output rows only the kept columns of X are fetched and multiplied (Section 3.1: only the
// non-zero columns of a block take part; Section 4.4: compact storage saves computation).
//
// Operands.  Per row-block the product is  Y[tile, block] = X[tile, kept columns] . vals^T  with
// 128 tokens as the M side of a tcgen05.mma, the d output rows as its N side and the kept columns
// as K.  Single columns of a row-major X are 2-byte pieces, useless for 16-byte copies, so the
// activations are taken TRANSPOSED, XT [k_in, tokens]: a kept column is then a contiguous row of
// 128 tokens (256 bytes), and TMA row gathers (tile::gather4: four rows of a 2-D tensor per
// instruction, box one row high) bring the kept rows straight into the tensor core's "MN-major"
// operand layout (8-row atoms of 64 tokens x 8 columns, 128-byte swizzle).  (A first version
// gathered with 16-byte cp.async copies; the load/store unit's limit on requests in flight held
// it to about 13 bytes per clock per SM.)  The weight
// side comes from a gather plan made once per pruned matrix: per pipeline stage (64 kept columns)
// the d x 64 tile already in the K-major 128-byte-swizzled layout (one bulk copy lands it), the
// 64 column numbers, and a byte that says how many 16-column groups are real and whether the stage
// starts or ends a row-block.
//
// Kernel.  Persistent CTAs walk units of (128-token tile) x (run of consecutive row-blocks); the
// stages of such a run are consecutive in the plan, so the producers just stream them.
//   warps 0-3 : producers, warp w filling every fourth stage; lane = (64-token half, four rows): one
//               gather4 per lane per stage, completion bytes counted on the stage's mbarrier;
//               lane 0 also issues the bulk copy of the weight tile and hands the stage's byte on;
//   warp 4    : one lane issues tcgen05.mma (M=128, N=d, K=16) into one of two TMEM accumulators,
//               commits stage release and, at the end of a row-block, accumulator ready;
//   warps 5-8 : epilogue; each warp reads its 32 TMEM lanes (tokens), adds bias, optional GELU,
//               rounds to bf16 and stores its row's d outputs (2 d contiguous bytes).
// Every wait is bounded; on expiry the role records BSP_ERR_TIMEOUT and leaves its loop.
//
// What bounds it: every gathered element crosses L2 -> shared memory once per row-block and feeds
// only d multiply-adds per token, so the operand traffic per flop is 1/d of a byte: the kernel
// pays off for tall blocks and high compression, where the zero-expanded dense route spends its
// time multiplying zeros.
#include "bsp_tc.cuh"

namespace bsp {

int check_linear_args(const void* a, const void* b, const void* c, int n_out, int k_in, int block,
                      const void* X, int tokens, int ldx, int act, const void* Y, int ldy);

using namespace tc;

namespace {

constexpr int kGThreads = 288;              // 4 producer warps, MMA warp, 4 epilogue warps
constexpr int kGStageK = 64;                // kept columns per pipeline stage
constexpr int kGStageA = kGStageK * kBlockM * 2;   // 16 KB: 64 rows of 128 tokens
constexpr int kGQueue = 12;                 // a producer warp loads its column numbers up to this many stages ahead
constexpr int kGPrefetch = kGQueue;         // the plan's column array is padded by this many stages

template <int D>
struct GatherCfg {
  static constexpr int kStageB = D * 128;                       // d rows of 64 bf16
  static constexpr int kStage = kGStageA + kStageB;
  static constexpr int kFixed = 1024 /*alignment slack*/ + 512 /*barriers, stage bytes*/;
  static constexpr int kStagesRaw = (kSmemLimit - kFixed) / kStage;
  static constexpr int kStages = kStagesRaw > 12 ? 12 : kStagesRaw;
  static constexpr int kTmemCols = 2 * D < 32 ? 32 : 2 * D;     // 32, 64, 128, 256
  static constexpr int kSmemBytes = kStages * kStage + kFixed;
};

// Layout of a gather plan in device memory (all regions 256-byte aligned):
//   soff  int32 [n_blocks + 1]   first stage of every row-block
//   meta  uint8 [stages]         bits 0-2: real 16-column groups (1..4), bit 4: first stage of its
//                                row-block, bit 5: last stage
//   cols  int16 [stages][64]     column of X for row r of the stage; -1 = zero row (padding inside a
//                                real group), -2 = beyond the real groups (not loaded, not multiplied)
//   tiles bf16  [stages][d][64]  weight tile, row n at byte n*128, 16-byte chunk c at (c ^ (n & 7))
struct GatherLayout {
  size_t soff_off, meta_off, cols_off, tiles_off, total;
  long long max_stages;
};
inline GatherLayout gather_layout(int n_out, int k_in, int block) {
  GatherLayout L;
  const long long nb = n_out / block;
  L.max_stages = nb * ((k_in + kGStageK - 1) / kGStageK);      // every row-block has at least one stage
  if (L.max_stages < nb) L.max_stages = nb;
  L.soff_off = 0;
  L.meta_off = round_up(sizeof(int32_t) * static_cast<size_t>(nb + 1), 256);
  L.cols_off = L.meta_off + round_up(static_cast<size_t>(L.max_stages) + 256, 256);
  L.tiles_off = L.cols_off + round_up(static_cast<size_t>(L.max_stages + kGPrefetch + 1) * kGStageK * 2, 256);
  L.total = L.tiles_off + round_up(static_cast<size_t>(L.max_stages) * block * 128, 256);
  return L;
}

// ---- plan construction -------------------------------------------------------------------
// soff[b] = number of stages of the row-blocks before b (one CTA, a running block-wide scan).
__global__ void __launch_bounds__(1024)
gather_plan_scan_kernel(const int32_t* __restrict__ blk_ptr, int n_blocks, int32_t* __restrict__ soff) {
  __shared__ int s_warp[32];
  int running = 0;
  for (int b0 = 0; b0 < n_blocks; b0 += blockDim.x) {
    const int b = b0 + threadIdx.x;
    int mine = 0;
    if (b < n_blocks) {
      const int kc = blk_ptr[b + 1] - blk_ptr[b];
      mine = kc > 0 ? (kc + kGStageK - 1) / kGStageK : 1;
    }
    int total;
    const int before = running + block_exclusive_scan(mine, s_warp, &total);
    if (b < n_blocks) soff[b] = before;
    running += total;
  }
  if (threadIdx.x == 0) soff[n_blocks] = running;
}

// One CTA per row-block: meta bytes, permuted column numbers and swizzled weight tiles of its stages.
__global__ void __launch_bounds__(256)
gather_plan_fill_kernel(const int32_t* __restrict__ blk_ptr, const int32_t* __restrict__ idx,
                        const uint16_t* __restrict__ vals, int block, const int32_t* __restrict__ soff,
                        uint8_t* __restrict__ meta, int16_t* __restrict__ cols, uint16_t* __restrict__ tiles) {
  const int b = blockIdx.x;
  const int lo = blk_ptr[b], kc = blk_ptr[b + 1] - lo;
  const int g0 = soff[b], n_st = soff[b + 1] - g0;
  const uint16_t* tile = vals + static_cast<size_t>(block) * lo;        // [block][kc]
  for (int s = threadIdx.x; s < n_st; s += blockDim.x) {
    const int left = kc - s * kGStageK;                                  // real columns from this stage on
    int groups = left <= 0 ? 1 : (left >= kGStageK ? 4 : (left + 15) / 16);
    meta[g0 + s] = static_cast<uint8_t>(groups | (s == 0 ? 0x10 : 0) | (s == n_st - 1 ? 0x20 : 0));
  }
  for (int e = threadIdx.x; e < n_st * kGStageK; e += blockDim.x) {
    const int s = e / kGStageK, r = e % kGStageK;
    const int k = s * kGStageK + r;
    const int left = kc - s * kGStageK;
    const int groups = left <= 0 ? 1 : (left >= kGStageK ? 4 : (left + 15) / 16);
    int16_t c = -2;
    if (r < groups * 16) c = k < kc ? static_cast<int16_t>(idx[lo + k]) : static_cast<int16_t>(-1);
    cols[static_cast<size_t>(g0 + s) * kGStageK + r] = c;
  }
  // weight tiles: one thread per 16-byte chunk (8 columns of one row)
  const int chunks = n_st * block * 8;
  for (int e = threadIdx.x; e < chunks; e += blockDim.x) {
    const int s = e / (block * 8), rem = e % (block * 8);
    const int n = rem >> 3, ch = rem & 7;
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int k0 = s * kGStageK + ch * 8 + 2 * i;
      const uint32_t v0 = k0 < kc ? tile[static_cast<size_t>(n) * kc + k0] : 0u;
      const uint32_t v1 = k0 + 1 < kc ? tile[static_cast<size_t>(n) * kc + k0 + 1] : 0u;
      w[i] = v0 | (v1 << 16);
    }
    uint16_t* dst = tiles + (static_cast<size_t>(g0 + s) * block + n) * 64 + ((ch ^ (n & 7)) << 3);
    *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// ---- transposed copy ---------------------------------------------------------------------
// XT[c, r] = X[r, c] for a row-major bf16 matrix; 64 x 64 tiles through shared memory, 16-byte
// global accesses on both sides (rows and cols multiples of 8).
__global__ void __launch_bounds__(256)
transpose_kernel(const uint16_t* __restrict__ X, int rows, int cols, int ldx, uint16_t* __restrict__ XT, int ldxt) {
  __shared__ uint16_t s_t[64][66];
  const int r0 = blockIdx.y * 64, c0 = blockIdx.x * 64;
  for (int e = threadIdx.x; e < 512; e += 256) {
    const int r = e >> 3, q = e & 7;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (r0 + r < rows && c0 + q * 8 < cols) v = __ldg(reinterpret_cast<const uint4*>(X + static_cast<size_t>(r0 + r) * ldx + c0 + q * 8));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      s_t[r][q * 8 + 2 * i] = static_cast<uint16_t>(w[i] & 0xffffu);
      s_t[r][q * 8 + 2 * i + 1] = static_cast<uint16_t>(w[i] >> 16);
    }
  }
  __syncthreads();
  for (int e = threadIdx.x; e < 512; e += 256) {
    const int c = e >> 3, q = e & 7;             // output row c (a column of X), 8 source rows q*8..q*8+7
    if (c0 + c < cols && r0 + q * 8 < rows) {
      uint32_t w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        w[i] = static_cast<uint32_t>(s_t[q * 8 + 2 * i][c]) | (static_cast<uint32_t>(s_t[q * 8 + 2 * i + 1][c]) << 16);
      *reinterpret_cast<uint4*>(XT + static_cast<size_t>(c0 + c) * ldxt + r0 + q * 8) = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

// ---- the kernel --------------------------------------------------------------------------
struct GatherParams {
  const uint16_t* XT;
  int ldxt, tokens, n_out, k_in, act;
  const uint16_t* bias;
  uint16_t* Y;
  int ldy;
  int transposed;            // Y is [n_out, tokens] (leading dimension ldy spans the tokens)
  const int32_t* soff;
  const uint8_t* meta;
  const int16_t* cols;
  const uint16_t* tiles;
  int n_blocks, m_tiles, n_chunks, rb_per_chunk;
  int* status;
};

// MN-major operand tile with the 128-byte swizzle: 8-row atoms 1024 bytes apart along the
// contraction, the two 64-token halves of the tile 8 KB apart.
__device__ __forceinline__ uint64_t gather_desc_a(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3ffff) >> 4);
  d |= static_cast<uint64_t>((kGStageK * 128) >> 4) << 16;      // leading byte offset / 16
  d |= static_cast<uint64_t>(1024 >> 4) << 32;                   // stride byte offset / 16
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
// bf16 x bf16 -> float32, A MN-major (bit 15), B K-major, M = 128, N = d.
__host__ __device__ constexpr uint32_t gather_idesc(int d) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (static_cast<uint32_t>(d >> 3) << 17) |
         (static_cast<uint32_t>(kBlockM >> 4) << 24);
}
__device__ __forceinline__ void tmem_load_16cols(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}

template <int D>
__global__ void __launch_bounds__(kGThreads, 1)
linear_gather_kernel(const __grid_constant__ CUtensorMap map_xt, const __grid_constant__ GatherParams P) {
  using Cfg = GatherCfg<D>;
  constexpr int S = Cfg::kStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  // [S stages: A 16 KB, B D*128][mbarriers][stage bytes][TMEM base]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S * Cfg::kStage);
  // bars[0..S) full, [S..2S) empty, [2S..2S+2) accumulator full, [2S+2..2S+4) accumulator empty
  uint8_t* s_meta = reinterpret_cast<uint8_t*>(bars + 2 * S + 4);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(s_meta + 16);
  volatile uint32_t* timed_out = tmem_holder + 1;     // set by a role whose wait expired

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };
  auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * S + a); };
  auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * S + 2 + a); };

  if (threadIdx.x == 0) {
    *timed_out = 0u;
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_xt)) : "memory");
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(acc_full_bar(a), 1); mbar_init(acc_empty_bar(a), 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)),
                 "r"(static_cast<uint32_t>(Cfg::kTmemCols)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  const int total_units = P.m_tiles * P.n_chunks;

  if (warp < 4) {
    // ---------------------------------------------------------------- producers
    // Warp w fills the stages whose running number is w (mod 4).  Lane = (64-token half, group of
    // four consecutive rows): one TMA gather4 per lane brings four kept columns (rows of XT) x 64
    // tokens into the stage with the 128-byte swizzle.  A row number equal to k_in is out of range
    // and reads as zeros (padding rows); tokens beyond the end read as zeros too.
    const int half = lane >> 4, quad4 = lane & 15;
    const uint32_t dst_lane = static_cast<uint32_t>(half * (kGStageK * 128) + quad4 * 512);
    long long n0 = 0;                                // stages before this unit, over all units of this CTA
    bool ok = true;
    for (int unit = blockIdx.x; unit < total_units && ok; unit += gridDim.x) {
      const int m = unit / P.n_chunks, ch = unit - m * P.n_chunks;
      const int rb0 = ch * P.rb_per_chunk, rb1 = min(P.n_blocks, rb0 + P.rb_per_chunk);
      const int g_begin = __ldg(P.soff + rb0), g_end = __ldg(P.soff + rb1);
      const int x = m * kBlockM + half * 64;
      const int first = g_begin + static_cast<int>(((warp - n0) % 4 + 4) % 4);   // this warp's first stage of the unit
      // column numbers and stage bytes are loaded two of the warp's stages (eight stages) ahead
      uint2 cq[2];
      uint32_t mq[2];
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        cq[q] = __ldg(reinterpret_cast<const uint2*>(P.cols + static_cast<size_t>(first + 4 * q) * kGStageK + quad4 * 4));
        mq[q] = __ldg(P.meta + first + 4 * q);
      }
      for (int g0 = first; g0 < g_end && ok; g0 += 8) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const int g = g0 + 4 * q;
          if (g < g_end && ok) {
            const long long n = n0 + (g - g_begin);
            const int stage = static_cast<int>(n % S);
            const uint32_t phase = static_cast<uint32_t>((n / S) & 1);
            if (!mbar_wait(empty_bar(stage), phase ^ 1u, P.status)) { ok = false; }
            if (ok) {
              const uint2 cv = cq[q];
              const uint32_t mt = mq[q];
              cq[q] = __ldg(reinterpret_cast<const uint2*>(P.cols + static_cast<size_t>(g + 8) * kGStageK + quad4 * 4));
              mq[q] = __ldg(P.meta + g + 8);
              const uint32_t a_dst = smem_base + stage * Cfg::kStage;
              const int groups = static_cast<int>(mt & 7u);
              if (lane == 0) {
                s_meta[stage] = static_cast<uint8_t>(mt);
                mbar_arrive_expect_tx(full_bar(stage), static_cast<uint32_t>(groups * 16 * kBlockM * 2 + Cfg::kStageB));
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(a_dst + kGStageA), "l"(reinterpret_cast<uint64_t>(P.tiles + static_cast<size_t>(g) * D * 64)),
                               "r"(static_cast<uint32_t>(Cfg::kStageB)), "r"(full_bar(stage))
                             : "memory");
              }
              __syncwarp();
              if (quad4 * 4 < groups * 16) {
                int r[4];
                r[0] = static_cast<int16_t>(cv.x & 0xffffu);
                r[1] = static_cast<int16_t>(cv.x >> 16);
                r[2] = static_cast<int16_t>(cv.y & 0xffffu);
                r[3] = static_cast<int16_t>(cv.y >> 16);
#pragma unroll
                for (int i = 0; i < 4; ++i) r[i] = r[i] < 0 ? P.k_in : r[i];
                asm volatile(
                    "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes "
                    "[%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
                    ::"r"(a_dst + dst_lane), "l"(reinterpret_cast<uint64_t>(&map_xt)), "r"(x), "r"(r[0]), "r"(r[1]),
                      "r"(r[2]), "r"(r[3]), "r"(full_bar(stage))
                    : "memory");
              }
            }
          }
        }
      }
      n0 += g_end - g_begin;
    }
    if (!ok && lane == 0) record_timeout(P.status, timed_out);
  } else if (warp == 4) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = gather_idesc(D);
      int stage = 0;
      uint32_t phase = 0;
      uint32_t acc_phase[2] = {0u, 0u};
      int acc = 0;
      bool ok = true;
      for (int unit = blockIdx.x; unit < total_units && ok; unit += gridDim.x) {
        const int m = unit / P.n_chunks, ch = unit - m * P.n_chunks;
        const int rb0 = ch * P.rb_per_chunk, rb1 = min(P.n_blocks, rb0 + P.rb_per_chunk);
        const int g_begin = __ldg(P.soff + rb0), g_end = __ldg(P.soff + rb1);
        for (int g = g_begin; g < g_end; ++g) {
          if (!mbar_wait(full_bar(stage), phase, P.status)) { ok = false; break; }
          tcgen05_fence_after();
          const uint32_t mt = s_meta[stage];
          const int groups = static_cast<int>(mt & 7u);
          const bool first = (mt & 0x10u) != 0, last = (mt & 0x20u) != 0;
          if (first) {
            if (!mbar_wait(acc_empty_bar(acc), acc_phase[acc] ^ 1u, P.status)) { ok = false; break; }
            tcgen05_fence_after();
          }
          const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * D);
          const uint32_t a_addr = smem_base + stage * Cfg::kStage;
          const uint32_t b_addr = a_addr + kGStageA;
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            if (k < groups)
              tcgen05_mma_bf16(d_tmem, gather_desc_a(a_addr + k * 2048), smem_desc_sw128(b_addr + k * 32), idesc,
                               (first && k == 0) ? 0u : 1u);
          }
          tcgen05_commit(empty_bar(stage));
          if (last) {
            tcgen05_commit(acc_full_bar(acc));
            acc_phase[acc] ^= 1u;
            acc ^= 1;
          }
          if (++stage == S) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) record_timeout(P.status, timed_out);
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    const int quad = warp & 3;               // TMEM lanes [32*quad, 32*quad+32) belong to this warp
    uint32_t acc_phase[2] = {0u, 0u};
    int acc = 0;
    bool ok = true;
    for (int unit = blockIdx.x; unit < total_units && ok; unit += gridDim.x) {
      const int m = unit / P.n_chunks, ch = unit - m * P.n_chunks;
      const int rb0 = ch * P.rb_per_chunk, rb1 = min(P.n_blocks, rb0 + P.rb_per_chunk);
      const int t = m * kBlockM + quad * 32 + lane;
      uint16_t* yrow = P.Y + static_cast<size_t>(t) * P.ldy;
      for (int rb = rb0; rb < rb1; ++rb) {
        // the bias of this row-block first, so that its latency overlaps the wait for the accumulator
        uint4 bv[D / 8];
#pragma unroll
        for (int j = 0; j < D / 8; ++j) bv[j] = make_uint4(0u, 0u, 0u, 0u);
        if (P.bias != nullptr) {
          const uint4* bp = reinterpret_cast<const uint4*>(P.bias + static_cast<size_t>(rb) * D);
#pragma unroll
          for (int j = 0; j < D / 8; ++j) bv[j] = __ldg(bp + j);
        }
        if (!mbar_wait(acc_full_bar(acc), acc_phase[acc], P.status)) { ok = false; break; }
        tcgen05_fence_after();
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(acc * D);
        constexpr int kPiece = 16;
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += kPiece) {
          uint32_t v[16];
          tmem_load_16cols(taddr + c0, v);
          tmem_load_wait();
          if (c0 + kPiece >= D) {              // this warp's last read of the accumulator
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty_bar(acc));
          }
          const uint4 b0 = bv[c0 / 8], b1 = bv[c0 / 8 + 1];
          const uint32_t bw[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
          float f[16];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            f[2 * i] = __uint_as_float(v[2 * i]) + __uint_as_float(bw[i] << 16);
            f[2 * i + 1] = __uint_as_float(v[2 * i + 1]) + __uint_as_float(bw[i] & 0xffff0000u);
          }
          if (P.act == BSP_ACT_GELU) {
#pragma unroll
            for (int i = 0; i < 16; i += 2) gelu_erf_pair(f[i], f[i + 1]);
          }
          if (P.transposed) {
            // output row n = rb * D + c0 + i holds this thread's token in column t: the 32 lanes of a warp
            // write 64 contiguous bytes per output row
            if (t < P.tokens) {
              uint16_t* col = P.Y + (static_cast<size_t>(rb) * D + c0) * P.ldy + t;
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const uint32_t w = pack_bf16x2(f[2 * i], f[2 * i + 1]);
                col[static_cast<size_t>(2 * i) * P.ldy] = static_cast<uint16_t>(w & 0xffffu);
                col[static_cast<size_t>(2 * i + 1) * P.ldy] = static_cast<uint16_t>(w >> 16);
              }
            }
          } else if (t < P.tokens) {
            uint4* out = reinterpret_cast<uint4*>(yrow + static_cast<size_t>(rb) * D + c0);
            out[0] = make_uint4(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]), pack_bf16x2(f[4], f[5]), pack_bf16x2(f[6], f[7]));
            out[1] = make_uint4(pack_bf16x2(f[8], f[9]), pack_bf16x2(f[10], f[11]), pack_bf16x2(f[12], f[13]), pack_bf16x2(f[14], f[15]));
          }
        }
        acc_phase[acc] ^= 1u;
        acc ^= 1;
      }
    }
    if (!ok && lane == 0) record_timeout(P.status, timed_out);
  }

  tcgen05_fence_before();
  __syncthreads();
  quiet_period(timed_out);
  if (warp == 4) {
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(static_cast<uint32_t>(Cfg::kTmemCols)) : "memory");
  }
}

template <int D>
int launch_gather(TcDevice* dev, int slot, const GatherParams& P, cudaStream_t s) {
  using Cfg = GatherCfg<D>;
  static_assert(Cfg::kStages >= 4, "pipeline too shallow");
  static bool attr_set[64] = {};
  int device = 0;
  BSP_CUDA_TRY(cudaGetDevice(&device));
  if (device < 0 || device >= 64) return BSP_ERR_CUDA;
  if (!attr_set[device]) {
    BSP_CUDA_TRY(cudaFuncSetAttribute(linear_gather_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
    attr_set[device] = true;
  }
  (void)slot;
  CUtensorMap map_xt;      // XT as [k_in rows, tokens]; box = one row of 64 tokens, 128-byte swizzle, zeros out of range
  // (no L2 promotion: a gathered row is 128 bytes, and fetching 256 would read every line twice)
  if (!make_map(&map_xt, P.XT, P.tokens, P.k_in, P.ldxt, 1, 64, CU_TENSOR_MAP_L2_PROMOTION_L2_128B)) return BSP_ERR_CUDA;
  const int units = P.m_tiles * P.n_chunks;
  const int grid = units < dev->sms ? units : dev->sms;
  linear_gather_kernel<D><<<grid, kGThreads, Cfg::kSmemBytes, s>>>(map_xt, P);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

bool gather_block_ok(int block) { return block == 16 || block == 32 || block == 64 || block == 128; }

}  // namespace
}  // namespace bsp

extern "C" int bsp_linear_gather_plan_bytes(int n_out, int k_in, int block, size_t* bytes) {
  using namespace bsp;
  if (n_out <= 0 || k_in <= 0 || block <= 0 || bytes == nullptr) return BSP_ERR_ARG;
  if (n_out % block) return BSP_ERR_SHAPE;
  if (!gather_block_ok(block) || k_in > 32767) return BSP_ERR_UNSUPPORTED;
  *bytes = gather_layout(n_out, k_in, block).total;
  return BSP_OK;
}

extern "C" int bsp_linear_gather_plan(const int32_t* blk_ptr, const int32_t* idx, const void* vals, int n_out,
                                      int k_in, int block, void* gplan, size_t gplan_bytes, void* stream) {
  using namespace bsp;
  if (blk_ptr == nullptr || idx == nullptr || vals == nullptr || gplan == nullptr) return BSP_ERR_ARG;
  size_t need;
  int st = bsp_linear_gather_plan_bytes(n_out, k_in, block, &need);
  if (st != BSP_OK) return st;
  if (!aligned_to(gplan, 256)) return BSP_ERR_ARG;
  if (gplan_bytes < need) return BSP_ERR_WORKSPACE;
  const GatherLayout L = gather_layout(n_out, k_in, block);
  char* base = static_cast<char*>(gplan);
  const int nb = n_out / block;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t* soff = reinterpret_cast<int32_t*>(base + L.soff_off);
  gather_plan_scan_kernel<<<1, 1024, 0, s>>>(blk_ptr, nb, soff);
  BSP_LAUNCH_CHECK();
  gather_plan_fill_kernel<<<nb, 256, 0, s>>>(blk_ptr, idx, static_cast<const uint16_t*>(vals), block, soff,
                                             reinterpret_cast<uint8_t*>(base + L.meta_off),
                                             reinterpret_cast<int16_t*>(base + L.cols_off),
                                             reinterpret_cast<uint16_t*>(base + L.tiles_off));
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

extern "C" int bsp_transpose(const void* X, int rows, int cols, int ldx, void* XT, int ldxt, void* stream) {
  using namespace bsp;
  if (X == nullptr || XT == nullptr || rows < 0 || cols <= 0) return BSP_ERR_ARG;
  if (ldx < cols || ldxt < rows) return BSP_ERR_SHAPE;
  if (rows % 8 || cols % 8 || ldx % 8 || ldxt % 8 || !aligned_to(X, 16) || !aligned_to(XT, 16)) return BSP_ERR_UNSUPPORTED;
  if (rows == 0) return BSP_OK;
  const dim3 grid((cols + 63) / 64, (rows + 63) / 64);
  if (grid.y > 65535) return BSP_ERR_UNSUPPORTED;
  transpose_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const uint16_t*>(X), rows, cols, ldx,
                                                                        static_cast<uint16_t*>(XT), ldxt);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

extern "C" int bsp_linear_gathered(const void* gplan, int n_out, int k_in, int block, const void* XT, int tokens,
                                   int ldxt, const void* bias, int act, void* Y, int ldy, void* stream) {
  return bsp_linear_gathered_ex(gplan, n_out, k_in, block, XT, tokens, ldxt, bias, act, Y, ldy, 0, stream);
}

extern "C" int bsp_linear_gathered_ex(const void* gplan, int n_out, int k_in, int block, const void* XT, int tokens,
                                      int ldxt, const void* bias, int act, void* Y, int ldy, int out_transposed,
                                      void* stream) {
  using namespace bsp;
  if (gplan == nullptr || XT == nullptr || Y == nullptr) return BSP_ERR_ARG;
  if (n_out <= 0 || k_in <= 0 || block <= 0 || tokens < 0) return BSP_ERR_ARG;
  if (act != BSP_ACT_NONE && act != BSP_ACT_GELU) return BSP_ERR_ARG;
  if (n_out % block) return BSP_ERR_SHAPE;
  if (ldxt < tokens || ldy < (out_transposed ? tokens : n_out)) return BSP_ERR_SHAPE;
  if (!gather_block_ok(block) || k_in > 32767) return BSP_ERR_UNSUPPORTED;
  if (!aligned_to(gplan, 256) || !aligned_to(XT, 16) || !aligned_to(Y, 16) || (bias != nullptr && !aligned_to(bias, 16)) ||
      tokens % 8 || ldxt % 8 || ldy % 8)
    return BSP_ERR_UNSUPPORTED;
  if (tokens == 0) return BSP_OK;
  TcDevice* dev = tc_device();
  if (dev == nullptr) return BSP_ERR_CUDA;
  const GatherLayout L = gather_layout(n_out, k_in, block);
  const char* base = static_cast<const char*>(gplan);
  GatherParams P;
  P.XT = static_cast<const uint16_t*>(XT);
  P.ldxt = ldxt;
  P.tokens = tokens;
  P.n_out = n_out;
  P.k_in = k_in;
  P.act = act;
  P.bias = static_cast<const uint16_t*>(bias);
  P.Y = static_cast<uint16_t*>(Y);
  P.ldy = ldy;
  P.transposed = out_transposed ? 1 : 0;
  P.soff = reinterpret_cast<const int32_t*>(base + L.soff_off);
  P.meta = reinterpret_cast<const uint8_t*>(base + L.meta_off);
  P.cols = reinterpret_cast<const int16_t*>(base + L.cols_off);
  P.tiles = reinterpret_cast<const uint16_t*>(base + L.tiles_off);
  P.n_blocks = n_out / block;
  P.m_tiles = (tokens + kBlockM - 1) / kBlockM;
  // runs of consecutive row-blocks: enough units for about six per SM, runs as long as that allows
  int n_chunks = (6 * dev->sms + P.m_tiles - 1) / P.m_tiles;
  if (n_chunks < 1) n_chunks = 1;
  if (n_chunks > P.n_blocks) n_chunks = P.n_blocks;
  P.rb_per_chunk = (P.n_blocks + n_chunks - 1) / n_chunks;
  P.n_chunks = (P.n_blocks + P.rb_per_chunk - 1) / P.rb_per_chunk;
  P.status = dev->status;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  switch (block) {
    case 16: return launch_gather<16>(dev, 0, P, s);
    case 32: return launch_gather<32>(dev, 1, P, s);
    case 64: return launch_gather<64>(dev, 2, P, s);
    default: return launch_gather<128>(dev, 3, P, s);
  }
}
