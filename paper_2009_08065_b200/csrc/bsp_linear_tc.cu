// bsp_linear / bsp_linear_plan / bsp_linear_planned: the pruned linear layer on the B200 tensor
// cores (tcgen05.mma with float32 accumulators in tensor memory, operands staged by TMA).
//
// Execution layout ("plan").  A row-block's kept-column list differs from its neighbours', and a
// tcgen05 operand tile addresses K in contiguous 16-byte pieces, so single columns cannot be
// picked from a resident X tile by the hardware.  Re-gathering X per row-block would move
// 2 bytes through shared memory per `block` multiply-adds, which caps the tensor pipe at about
// block/64 of its peak.  The plan therefore scatters the packed values back to their natural
// column positions, zero elsewhere: a [n_out, k_in] bf16 matrix that TMA can tile directly,
// with X read in its natural order and reused by a whole 128 x BN output tile.  The packed form
// stays the storage format; the plan is private scratch derived from it.
//
// Kernel.  Persistent CTAs (one per SM) walk output tiles of 128 tokens x BN outputs.
//   warp 0 (one lane): TMA producer, X tile [128 x 64] and W tile [BN x 64] per pipeline stage
//                      (128-byte swizzle), completion on an mbarrier;
//   warp 1 (one lane): issues tcgen05.mma (M=128, N=BN, K=16) into one of two TMEM accumulators
//                      and commits stage release / accumulator ready to mbarriers;
//   warps 2..9       : epilogue, two groups of four warps; group g takes the 32-column pieces of
//                      the tile with index = g (mod 2).  Each warp tcgen05.ld's its 32 TMEM lanes
//                      (= 32 tokens), adds bias, optional GELU, rounds to bf16, writes its rows
//                      into the group's swizzled staging buffer, and one thread hands the
//                      128 x 32 piece to a TMA store (full-line writes, tails clipped by the
//                      tensor map).  The epilogue runs concurrently with the next tile's main
//                      loop on the other accumulator.
// Every wait is bounded by a wall-clock deadline (bsp_set_wait_limit_ms); on expiry the role records
// BSP_ERR_TIMEOUT in the status word and leaves its loop, the other roles then time out on their
// own waits (the epilogue threads by a common vote), and the CTA waits a millisecond for whatever
// it still has in flight, frees its tensor memory and exits.
#include <mutex>
#include <cstring>

#include "bsp_tc.cuh"

namespace bsp {

int check_linear_args(const void* a, const void* b, const void* c, int n_out, int k_in, int block,
                      const void* X, int tokens, int ldx, int act, const void* Y, int ldy);
int launch_tc_pair(TcDevice* dev, const void* plan, const void* X, void* Y, int tokens, int n_out, int k_in, int act,
                   const void* bias, int ldx, int ldy, cudaStream_t s);

using namespace tc;

namespace {

// [0]: 0, or BSP_ERR_TIMEOUT once a bounded wait expired; [1]: a counter nothing ever bumps (self-test);
// [2..3]: the limit of one wait in nanoseconds; [4]: waits that ran out in the last self-test;
// [6..7]: how long its mbarrier wait lasted, nanoseconds
__device__ __align__(16) int g_linear_status[8];


struct LinearParams {
  int tokens, n_out, k_in, act;
  int plan_stable;      // the plan was complete before the kernel preceding this one in the stream began
  int transposed;       // the output is written as [n_out, tokens] (map_y describes that matrix)
  const uint16_t* bias;
  int* status;
};

// Epilogue groups of four warps (one warp per quarter of the TMEM lanes), two staging buffers each.
// Four groups with one buffer each (the same 32 KB; the exposed epilogue of a CTA's last tile then takes
// two pieces per group instead of four) were measured 1.5 us slower per four-GEMM layer at 4096 tokens:
// sixteen warps contend for the shared memory that the operand copies and the tensor core keep busy.
#ifndef BSP_TC_GROUPS
#define BSP_TC_GROUPS 2
#endif
constexpr int kGroups = BSP_TC_GROUPS;
constexpr int kEpiThreads = 128 * kGroups;
constexpr int kBufPerGroup = kEpiBuffers / kGroups;
static_assert(kGroups == 2 || kGroups == 4, "two or four epilogue groups");
constexpr int kWeightWarp = 2 + 4 * kGroups;            // the second TMA producer warp, for the weight tiles
constexpr int kThreadsTc = 32 * (kWeightWarp + 1);

// Named barriers of this kernel's epilogue: 5 + g among the 128 threads of group g, 3 and 4 among all of them.
__device__ __forceinline__ void tc_group_sync(int g) { asm volatile("bar.sync %0, 128;" ::"r"(5 + g) : "memory"); }
__device__ __forceinline__ void tc_epilogue_sync_all() { asm volatile("bar.sync 3, %0;" ::"n"(kEpiThreads) : "memory"); }
__device__ __forceinline__ bool tc_epilogue_all_ok(bool ok) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 p, %1, 0;\n\t"
      "barrier.cta.red.and.pred q, 4, %2, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r)
      : "r"(ok ? 1u : 0u), "n"(kEpiThreads)
      : "memory");
  return r != 0u;
}

template <int BN>
__global__ void __launch_bounds__(kThreadsTc, 1)
linear_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                 const __grid_constant__ CUtensorMap map_y, LinearParams P) {
  using Cfg = TileCfg<BN>;
  constexpr int S = Cfg::kStages;
  extern __shared__ uint8_t smem_raw[];
  // operand stages need 1024-byte alignment for the 128-byte swizzle pattern
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  // [S operand stages][2 epilogue staging buffers][bias, bf16, for two tiles][mbarriers, TMEM base]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S * Cfg::kStage + kEpiBytes + 2 * BN * 2);
  // bars[0..S) full, [S..2S) empty, [2S..2S+2) accumulator full, [2S+2..2S+4) accumulator empty
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 2 * S + 4);
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
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_x)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_w)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_y)) : "memory");
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 2); mbar_init(empty_bar(s), 1); }   // two producers arm a stage
    for (int a = 0; a < 2; ++a) { mbar_init(acc_full_bar(a), 1); mbar_init(acc_empty_bar(a), 4 * kGroups); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)),
                 "r"(static_cast<uint32_t>(Cfg::kTmemCols)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  // Programmatic dependent launch: everything above touched only this CTA's shared and tensor
  // memory and overlaps the tail of the previous kernel in the stream.  From here on the kernel
  // reads memory that kernel may have written (X, the plan), so wait for it to finish; and let
  // the next kernel in the stream start its own prologue as soon as SMs become free.  When the
  // caller vouches that the plan is older than the previous kernel, the weight producer does not
  // wait: its first tiles are on their way while the previous kernel finishes writing X.
  if (!(P.plan_stable && warp == kWeightWarp)) asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const int m_tiles = (P.tokens + kBlockM - 1) / kBlockM;
  const int n_tiles = (P.n_out + BN - 1) / BN;
  const int total_tiles = m_tiles * n_tiles;
  const int k_blocks = (P.k_in + kBlockK - 1) / kBlockK;

  if (warp == 0 && lane == 0) {
    // ---------------------------------------------------------------- TMA producer of the X tiles
    // (the two operands of a stage are issued by two warps, this one and the last one, so neither waits
    // behind the other's copy)
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int m0 = (tile / n_tiles) * kBlockM;
      for (int kb = 0; kb < k_blocks; ++kb) {
        if (!mbar_wait(empty_bar(stage), phase ^ 1u, P.status)) { ok = false; break; }
        const uint32_t a_dst = smem_base + stage * Cfg::kStage;
        mbar_arrive_expect_tx(full_bar(stage), Cfg::kStageA);
        tma_load_2d(a_dst, &map_x, kb * kBlockK, m0, full_bar(stage));
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
    }
    if (!ok) record_timeout(P.status, timed_out);
  } else if (warp == kWeightWarp && lane == 0) {
    // ---------------------------------------------------------------- TMA producer of the weight tiles
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int n0 = (tile % n_tiles) * BN;
      for (int kb = 0; kb < k_blocks; ++kb) {
        if (!mbar_wait(empty_bar(stage), phase ^ 1u, P.status)) { ok = false; break; }
        mbar_arrive_expect_tx(full_bar(stage), Cfg::kStageB);
        tma_load_2d(smem_base + stage * Cfg::kStage + Cfg::kStageA, &map_w, kb * kBlockK, n0, full_bar(stage));
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
    }
    if (!ok) record_timeout(P.status, timed_out);
  } else if (warp == 1 && lane == 0) {
    // ---------------------------------------------------------------- MMA issuer
    constexpr uint32_t idesc = instr_desc_bf16(BN);
    int stage = 0;
    uint32_t phase = 0;
    uint32_t acc_phase[2] = {0u, 0u};
    int acc = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      if (!mbar_wait(acc_empty_bar(acc), acc_phase[acc] ^ 1u, P.status)) { ok = false; break; }
      tcgen05_fence_after();
      const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
      for (int kb = 0; kb < k_blocks; ++kb) {
        if (!mbar_wait(full_bar(stage), phase, P.status)) { ok = false; break; }
        tcgen05_fence_after();
        const uint32_t a_addr = smem_base + stage * Cfg::kStage;
        const uint32_t b_addr = a_addr + Cfg::kStageA;
#pragma unroll
        for (int k = 0; k < kBlockK / kUmmaK; ++k) {
          const uint64_t a_desc = smem_desc_sw128(a_addr + k * kUmmaK * 2);
          const uint64_t b_desc = smem_desc_sw128(b_addr + k * kUmmaK * 2);
          tcgen05_mma_bf16(d_tmem, a_desc, b_desc, idesc, (kb | k) != 0 ? 1u : 0u);
        }
        tcgen05_commit(empty_bar(stage));  // stage reusable once these MMAs have read it
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
      if (!ok) break;
      tcgen05_commit(acc_full_bar(acc));   // accumulator complete
      acc_phase[acc] ^= 1u;
      acc ^= 1;
    }
    if (!ok) record_timeout(P.status, timed_out);
  } else if (warp >= 2 && warp < kWeightWarp) {
    // ---------------------------------------------------------------- epilogue
    const int group = (warp - 2) >> 2;
    const int quad = warp & 3;               // TMEM lanes [32*quad, 32*quad+32) belong to this warp
    const int row = quad * 32 + lane;        // token row of this thread inside the tile
    const int epi_tid = threadIdx.x - 64;    // index among the epilogue threads
    const bool issuer = (epi_tid & 127) == 0;  // the thread of each group that owns its TMA stores
    const uint32_t buf0 = smem_base + S * Cfg::kStage + group * kBufPerGroup * kEpiStage;   // this group's staging buffers
    uint32_t my_piece = 0;                   // pieces staged by this group so far: selects the buffer
    uint16_t* s_bias = reinterpret_cast<uint16_t*>(smem + S * Cfg::kStage + kEpiBytes);  // [2][BN] bf16
    const uint32_t row_off = static_cast<uint32_t>(row) * 64u;
    const uint32_t row_xor = static_cast<uint32_t>((row >> 1) & 3);
    uint32_t acc_phase[2] = {0u, 0u};
    int acc = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int m0 = (tile / n_tiles) * kBlockM, n0 = (tile % n_tiles) * BN;
      // Bias of this tile's columns, in the half of s_bias that belongs to this accumulator.  The
      // other group can lag by at most one tile (it has to reach the barrier below for this tile),
      // so the values it may still be reading are in the other half.
      for (int c = epi_tid; c < BN; c += kEpiThreads)
        s_bias[acc * BN + c] = (P.bias != nullptr && n0 + c < P.n_out) ? __ldg(P.bias + n0 + c) : static_cast<uint16_t>(0);
      tc_epilogue_sync_all();
      // all epilogue threads take the same decision, so nobody is left alone at a named barrier below
      if (!tc_epilogue_all_ok(mbar_wait(acc_full_bar(acc), acc_phase[acc], P.status))) { ok = false; break; }
      tcgen05_fence_after();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(acc * BN);
      const int pieces = (min(BN, P.n_out - n0) + kEpiCols - 1) / kEpiCols;
      bool released = false;
#pragma unroll 1
      for (int pc = group; pc < pieces; pc += kGroups) {
        const int c0 = pc * kEpiCols;
        const uint32_t buf = buf0 + (my_piece % kBufPerGroup) * kEpiStage;
        ++my_piece;
        EpiloguePiece piece;
        piece_load(taddr + c0, smem_u32(s_bias + acc * BN + c0), piece);
        if (issuer) tma_store_wait_read<kBufPerGroup - 1>();   // the store that last used this buffer has read it
        tc_group_sync(group);
        if (pc + kGroups >= pieces) {        // this warp's last read of the accumulator
          tcgen05_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(acc_empty_bar(acc));
          released = true;
        }
        if (P.transposed) piece_store_transposed(piece, P.act, buf, row);
        else piece_store(piece, P.act, buf + row_off, row_xor);
        fence_async_smem();                  // make the staged piece visible to the TMA engine
        tc_group_sync(group);
        if (issuer) {
          // rows beyond `tokens` / columns beyond `n_out` are clipped by the tensor map
          if (P.transposed) tma_store_2d(&map_y, m0, n0 + c0, buf);
          else tma_store_2d(&map_y, n0 + c0, m0, buf);
          tma_store_commit();
        }
      }
      if (!released) {                       // a group without a piece in this tile still releases the accumulator
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty_bar(acc));
      }
      acc_phase[acc] ^= 1u;
      acc ^= 1;
    }
    if (issuer) tma_store_wait_read<0>();   // shared memory must outlive the reads; the writes complete with the grid
    if (!ok && lane == 0) record_timeout(P.status, timed_out);
  }

  tcgen05_fence_before();
  __syncthreads();
  quiet_period(timed_out);
  if (warp == 1) {
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(static_cast<uint32_t>(Cfg::kTmemCols)) : "memory");
  }
}

// Self-test of the bail-out path: one CTA sets up what the tensor-core kernels set up (an mbarrier,
// tensor memory), then two of its threads wait through the same helpers on a barrier and on a
// counter that nothing ever signals.  Both waits run out at the configured limit, the roles record
// it, the CTA sits out the quiet period, frees its tensor memory and returns by itself.
__global__ void __launch_bounds__(128, 1) wait_selftest_kernel(int* status) {
  __shared__ __align__(8) uint64_t s_bar;
  __shared__ uint32_t s_tmem[2];
  volatile uint32_t* timed_out = s_tmem + 1;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    *timed_out = 0u;
    status[4] = 0;
    mbar_init(smem_u32(&s_bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(32u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = s_tmem[0];
  if (warp == 0 && lane == 0) {
    const unsigned long long t0 = global_timer_ns();
    if (!mbar_wait(smem_u32(&s_bar), 0u, status)) {
      record_timeout(status, timed_out);
      atomicAdd(status + 4, 1);
    }
    const unsigned long long dt = global_timer_ns() - t0;
    *reinterpret_cast<volatile unsigned long long*>(status + 6) = dt;
  } else if (warp == 2 && lane == 0) {
    if (!wait_counter(status + 1, 1, status)) {
      record_timeout(status, timed_out);
      atomicAdd(status + 4, 1);
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  quiet_period(timed_out);
  if (warp == 1) {
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(32u) : "memory");
  }
}

// Plan: put the packed tiles of one row-block back at their natural column positions, zero
// elsewhere.  grid = (row-blocks, row splits); one thread produces 8 adjacent columns of a row
// (one 16-byte store), looking the columns up in a shared column -> kept-position table.
__global__ void __launch_bounds__(256)
plan_expand_kernel(const int32_t* __restrict__ blk_ptr, const int32_t* __restrict__ idx,
                   const uint16_t* __restrict__ vals, int k_in, int block, uint16_t* __restrict__ Wx) {
  extern __shared__ int16_t s_pos[];      // column -> position in the kept list, or -1 (k_in < 32768)
  const int b = blockIdx.x;
  const int lo = blk_ptr[b], kc = blk_ptr[b + 1] - lo;
  for (int k = threadIdx.x; k < k_in; k += blockDim.x) s_pos[k] = -1;
  __syncthreads();
  for (int j = threadIdx.x; j < kc; j += blockDim.x) s_pos[idx[lo + j]] = static_cast<int16_t>(j);
  __syncthreads();
  const uint16_t* tile = vals + static_cast<size_t>(block) * lo;
  const int rows_per = (block + gridDim.y - 1) / gridDim.y;
  const int r_lo = blockIdx.y * rows_per;
  const int r_hi = min(block, r_lo + rows_per);
  const int chunks = k_in >> 3;
  for (int e = threadIdx.x; e < (r_hi - r_lo) * chunks; e += blockDim.x) {
    const int r = r_lo + e / chunks, q = e % chunks;
    const uint4 pos4 = *reinterpret_cast<const uint4*>(s_pos + (q << 3));
    const uint32_t pw[4] = {pos4.x, pos4.y, pos4.z, pos4.w};
    const uint16_t* trow = tile + static_cast<size_t>(r) * kc;
    uint32_t out[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int p0 = static_cast<int16_t>(pw[i] & 0xffffu), p1 = static_cast<int16_t>(pw[i] >> 16);
      const uint32_t v0 = p0 >= 0 ? __ldg(trow + p0) : 0u;
      const uint32_t v1 = p1 >= 0 ? __ldg(trow + p1) : 0u;
      out[i] = v0 | (v1 << 16);
    }
    *reinterpret_cast<uint4*>(Wx + (static_cast<size_t>(b) * block + r) * k_in + (q << 3)) =
        make_uint4(out[0], out[1], out[2], out[3]);
  }
}

// Plan from the orientation-R packed form (vertical strips of h columns, kept ROWS per strip,
// tiles [kc][h]): every kept row segment goes back to its place; the plan is zeroed beforehand.
__global__ void __launch_bounds__(256)
plan_expand_r_kernel(const int32_t* __restrict__ blk_ptr, const int32_t* __restrict__ row_idx,
                     const uint16_t* __restrict__ vals, int k_in, int h, uint16_t* __restrict__ Wx) {
  const int a = blockIdx.x;                       // strip
  const int lo = blk_ptr[a], kc = blk_ptr[a + 1] - lo;
  const uint16_t* tile = vals + static_cast<size_t>(h) * lo;
  for (int e = threadIdx.x; e < kc * h; e += blockDim.x) {
    const int p = e / h, c = e - p * h;
    Wx[static_cast<size_t>(row_idx[lo + p]) * k_in + static_cast<size_t>(a) * h + c] = tile[e];
  }
}

// Transposed plan from the orientation-C packed form: PT[k, n] = (W * Mask)[n, k], for the product
// dX = dY (W * Mask).  One CTA per row-block; consecutive threads take consecutive rows r of the
// block, so the 2-byte stores of one kept column are contiguous.  The plan is zeroed beforehand.
__global__ void __launch_bounds__(256)
plan_expand_t_kernel(const int32_t* __restrict__ blk_ptr, const int32_t* __restrict__ idx,
                     const uint16_t* __restrict__ vals, int n_out, int block, uint16_t* __restrict__ PT) {
  const int b = blockIdx.x;
  const int lo = blk_ptr[b], kc = blk_ptr[b + 1] - lo;
  const uint16_t* tile = vals + static_cast<size_t>(block) * lo;
  for (int e = threadIdx.x; e < kc * block; e += blockDim.x) {
    const int j = e / block, r = e - j * block;
    PT[static_cast<size_t>(idx[lo + j]) * n_out + static_cast<size_t>(b) * block + r] = tile[static_cast<size_t>(r) * kc + j];
  }
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
}  // namespace
// Output-tile width: fewest (waves x per-tile cost) over the candidates.  A 64-deep stage of the main
// loop was measured at about 460 / 515 / 545 / 640 cycles for tiles 64 / 128 / 192 / 256 outputs wide (the
// activation tile and the latencies are the same whatever the width), which 440 + width models.
int choose_bn(int tokens, int n_out, int sms) {
  const int cands[4] = {256, 192, 128, 64};
  long long best = -1;
  int best_bn = 128;
  const long long m_tiles = (tokens + kBlockM - 1) / kBlockM;
  for (int c = 0; c < 4; ++c) {
    const int bn = cands[c];
    const long long tiles = m_tiles * ((n_out + bn - 1) / bn);
    const long long waves = (tiles + sms - 1) / sms;
    const long long cost = waves * (bn + 440);
    if (best < 0 || cost < best) { best = cost; best_bn = bn; }
  }
  return best_bn;
}
namespace {

template <int BN>
int launch_tc(TcDevice* dev, int slot, const void* plan, const void* X, void* Y, const LinearParams& P, int ldx,
              int ldy, cudaStream_t s) {
  using Cfg = TileCfg<BN>;
  static_assert(Cfg::kStages >= 3, "pipeline too shallow");
  static_assert(BN % kEpiCols == 0, "tile width must be a multiple of the epilogue piece");
  CUtensorMap map_x, map_w, map_y;
  if (!make_map(&map_x, X, P.k_in, P.tokens, ldx, kBlockM)) return BSP_ERR_CUDA;
  if (!make_map(&map_w, plan, P.k_in, P.n_out, P.k_in, BN)) return BSP_ERR_CUDA;
  if (P.transposed) {     // Y is [n_out, tokens]: pieces of 32 output rows x 128 tokens
    if (!make_map(&map_y, Y, P.tokens, P.n_out, ldy, kEpiCols, kBlockM)) return BSP_ERR_CUDA;
  } else if (!make_map(&map_y, Y, P.n_out, P.tokens, ldy, kBlockM, kEpiCols)) {
    return BSP_ERR_CUDA;
  }
  if (!dev->attr_set[slot]) {
    BSP_CUDA_TRY(cudaFuncSetAttribute(linear_tc_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
    dev->attr_set[slot] = true;
  }
  const int m_tiles = (P.tokens + kBlockM - 1) / kBlockM;
  const int n_tiles = (P.n_out + BN - 1) / BN;
  const int tiles = m_tiles * n_tiles;
  const int grid = tiles < dev->sms ? tiles : dev->sms;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreadsTc);
  cfg.dynamicSmemBytes = Cfg::kSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // start while the previous kernel drains
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  BSP_CUDA_TRY(cudaLaunchKernelEx(&cfg, linear_tc_kernel<BN>, map_x, map_w, map_y, P));
  return BSP_OK;
}

bool tc_path_ok(const void* plan, int n_out, int k_in, const void* X, int ldx, const void* Y, int ldy) {
  return aligned_to(plan, 16) && aligned_to(X, 16) && aligned_to(Y, 16) && k_in % 8 == 0 && ldx % 8 == 0 &&
         ldy % 8 == 0 && n_out % 8 == 0 && k_in <= 12288;
}

}  // namespace

TcDevice* tc_device() {
  static TcDevice info[64];
  static std::mutex guard;             // first calls from several host threads must not race on the set-up
  std::lock_guard<std::mutex> lock(guard);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  TcDevice& d = info[dev];
  if (d.sms == 0) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return nullptr;
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_linear_status) != cudaSuccess) return nullptr;
    const unsigned long long limit = kDefaultWaitLimitNs;
    int init[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    memcpy(&init[2], &limit, sizeof(limit));
    if (cudaMemcpy(p, init, sizeof(init), cudaMemcpyHostToDevice) != cudaSuccess) return nullptr;
    d.status = static_cast<int*>(p);
    d.sms = sms;
  }
  return &d;
}

}  // namespace bsp

extern "C" int bsp_linear_plan_bytes(int n_out, int k_in, int block, size_t* bytes) {
  if (n_out <= 0 || k_in <= 0 || block <= 0 || bytes == nullptr) return BSP_ERR_ARG;
  if (n_out % block) return BSP_ERR_SHAPE;
  *bytes = bsp::round_up(static_cast<size_t>(n_out) * k_in * 2, 256);
  return BSP_OK;
}

extern "C" int bsp_linear_plan(const int32_t* blk_ptr, const int32_t* idx, const void* vals, int n_out,
                               int k_in, int block, void* plan, size_t plan_bytes, void* stream) {
  using namespace bsp;
  if (blk_ptr == nullptr || idx == nullptr || vals == nullptr || plan == nullptr) return BSP_ERR_ARG;
  size_t need;
  int st = bsp_linear_plan_bytes(n_out, k_in, block, &need);
  if (st != BSP_OK) return st;
  if (!aligned_to(plan, 256)) return BSP_ERR_ARG;
  if (plan_bytes < need) return BSP_ERR_WORKSPACE;
  if (k_in > 12288) return BSP_ERR_UNSUPPORTED;
  if (k_in % 8) return BSP_ERR_UNSUPPORTED;
  const int splits = block >= 4 ? 4 : 1;
  plan_expand_kernel<<<dim3(n_out / block, splits), 256, sizeof(int16_t) * k_in, static_cast<cudaStream_t>(stream)>>>(
      blk_ptr, idx, static_cast<const uint16_t*>(vals), k_in, block, static_cast<uint16_t*>(plan));
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

extern "C" int bsp_linear_plan_r(const int32_t* blk_ptr, const int32_t* row_idx, const void* vals, int n_out,
                                 int k_in, int block, void* plan, size_t plan_bytes, void* stream) {
  using namespace bsp;
  if (blk_ptr == nullptr || row_idx == nullptr || vals == nullptr || plan == nullptr) return BSP_ERR_ARG;
  if (n_out <= 0 || k_in <= 0 || block <= 0) return BSP_ERR_ARG;
  if (k_in % block) return BSP_ERR_SHAPE;
  if (!aligned_to(plan, 256)) return BSP_ERR_ARG;
  const size_t need = round_up(static_cast<size_t>(n_out) * k_in * 2, 256);
  if (plan_bytes < need) return BSP_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  BSP_CUDA_TRY(cudaMemsetAsync(plan, 0, static_cast<size_t>(n_out) * k_in * 2, s));
  plan_expand_r_kernel<<<k_in / block, 256, 0, s>>>(blk_ptr, row_idx, static_cast<const uint16_t*>(vals), k_in, block,
                                                   static_cast<uint16_t*>(plan));
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

extern "C" int bsp_linear_plan_t(const int32_t* blk_ptr, const int32_t* idx, const void* vals, int n_out, int k_in,
                                 int block, void* plan_t, size_t plan_bytes, void* stream) {
  using namespace bsp;
  if (blk_ptr == nullptr || idx == nullptr || vals == nullptr || plan_t == nullptr) return BSP_ERR_ARG;
  size_t need;
  int st = bsp_linear_plan_bytes(n_out, k_in, block, &need);
  if (st != BSP_OK) return st;
  if (!aligned_to(plan_t, 256)) return BSP_ERR_ARG;
  if (plan_bytes < need) return BSP_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  BSP_CUDA_TRY(cudaMemsetAsync(plan_t, 0, static_cast<size_t>(n_out) * k_in * 2, s));
  plan_expand_t_kernel<<<n_out / block, 256, 0, s>>>(blk_ptr, idx, static_cast<const uint16_t*>(vals), n_out, block,
                                                     static_cast<uint16_t*>(plan_t));
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

extern "C" int bsp_linear_planned_ex(const void* plan, int n_out, int k_in, int block, const void* X, int tokens,
                                     int ldx, const void* bias, int act, void* Y, int ldy, int algo, void* stream) {
  using namespace bsp;
  const int algo_flags = algo & ~0xff;
  algo &= 0xff;
  if (algo < BSP_LINEAR_AUTO || algo > BSP_LINEAR_CTA_PAIR || (algo_flags & ~(BSP_LINEAR_PLAN_STABLE | BSP_LINEAR_OUT_TRANSPOSED)))
    return BSP_ERR_ARG;
  const bool transposed = (algo_flags & BSP_LINEAR_OUT_TRANSPOSED) != 0;
  if (transposed && algo == BSP_LINEAR_CTA_PAIR) return BSP_ERR_UNSUPPORTED;     // only the one-CTA kernel writes transposed
  // (a transposed output is [n_out, tokens]: its leading dimension spans the tokens)
  int st = check_linear_args(plan, plan, plan, n_out, k_in, block, X, tokens, ldx, act, Y, transposed ? n_out : ldy);
  if (st != BSP_OK) return st;
  if (transposed && ldy < tokens) return BSP_ERR_SHAPE;
  if (!tc_path_ok(plan, n_out, k_in, X, ldx, Y, ldy)) return BSP_ERR_UNSUPPORTED;
  if (tokens == 0) return BSP_OK;
  TcDevice* dev = tc_device();
  if (dev == nullptr) return BSP_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // Measured on B200, single launches after an L2 flush: without GELU the CTA-pair kernel is level or ahead
  // from about 1.25 x #SM pair-tiles on (8192 tokens x 2304 outputs: 3 %; 16384 x 768: 3-9 %; 32768 tokens: 4-11 %;
  // a 1024 x 4096 weight at 16384 tokens: 30 %, the one-CTA kernel's last wave being half empty there) and behind
  // below that (one encoder layer at 4096 tokens: +0 to +4 us per launch; 8192 x 768 x 768: +13 %), where its
  // longer start-up shows.  With GELU the epilogue is the longer side of a tile and the two are level on average
  // (0.92-1.05 over six shapes), so those launches stay with the one-CTA kernel.
  const long long pair_tiles = static_cast<long long>((tokens + 255) / 256) * ((n_out + 255) / 256);
  const bool pair = algo == BSP_LINEAR_CTA_PAIR ||
                    (algo == BSP_LINEAR_AUTO && 4 * pair_tiles >= 5LL * dev->sms && act == BSP_ACT_NONE && !transposed);
  if (pair) return launch_tc_pair(dev, plan, X, Y, tokens, n_out, k_in, act, bias, ldx, ldy, s);
  LinearParams P{tokens, n_out, k_in, act, (algo_flags & BSP_LINEAR_PLAN_STABLE) ? 1 : 0, transposed ? 1 : 0,
                 static_cast<const uint16_t*>(bias), dev->status};
  switch (choose_bn(tokens, n_out, dev->sms)) {
    case 256: return launch_tc<256>(dev, 0, plan, X, Y, P, ldx, ldy, s);
    case 192: return launch_tc<192>(dev, 1, plan, X, Y, P, ldx, ldy, s);
    case 128: return launch_tc<128>(dev, 2, plan, X, Y, P, ldx, ldy, s);
    default: return launch_tc<64>(dev, 3, plan, X, Y, P, ldx, ldy, s);
  }
}

extern "C" int bsp_linear_planned(const void* plan, int n_out, int k_in, int block, const void* X, int tokens,
                                  int ldx, const void* bias, int act, void* Y, int ldy, void* stream) {
  return bsp_linear_planned_ex(plan, n_out, k_in, block, X, tokens, ldx, bias, act, Y, ldy, BSP_LINEAR_AUTO, stream);
}

extern "C" int bsp_linear(const int32_t* blk_ptr, const int32_t* idx, const void* vals, int n_out, int k_in,
                          int block, const void* X, int tokens, int ldx, const void* bias, int act, void* Y,
                          int ldy, void* ws, size_t ws_bytes, void* stream) {
  using namespace bsp;
  int st = check_linear_args(blk_ptr, idx, vals, n_out, k_in, block, X, tokens, ldx, act, Y, ldy);
  if (st != BSP_OK) return st;
  if (ws == nullptr || !aligned_to(ws, 256) || !tc_path_ok(ws, n_out, k_in, X, ldx, Y, ldy))
    return bsp_linear_cuda_core(blk_ptr, idx, vals, n_out, k_in, block, X, tokens, ldx, bias, act, Y, ldy, stream);
  st = bsp_linear_plan(blk_ptr, idx, vals, n_out, k_in, block, ws, ws_bytes, stream);
  if (st != BSP_OK) return st;
  return bsp_linear_planned(ws, n_out, k_in, block, X, tokens, ldx, bias, act, Y, ldy, stream);
}

extern "C" int bsp_set_wait_limit_ms(int ms) {
  using namespace bsp;
  if (ms < 1 || ms > 600000) return BSP_ERR_ARG;
  TcDevice* dev = tc_device();
  if (dev == nullptr) return BSP_ERR_CUDA;
  const unsigned long long ns = static_cast<unsigned long long>(ms) * 1000000ull;
  BSP_CUDA_TRY(cudaDeviceSynchronize());         // kernels in flight keep the limit they started with
  BSP_CUDA_TRY(cudaMemcpy(dev->status + 2, &ns, sizeof(ns), cudaMemcpyHostToDevice));
  return BSP_OK;
}

extern "C" int bsp_wait_selftest(int* expired, long long* waited_ns, void* stream) {
  using namespace bsp;
  TcDevice* dev = tc_device();
  if (dev == nullptr) return BSP_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  wait_selftest_kernel<<<1, 128, 0, s>>>(dev->status);
  BSP_LAUNCH_CHECK();
  int report[4] = {0, 0, 0, 0};
  BSP_CUDA_TRY(cudaMemcpyAsync(report, dev->status + 4, sizeof(report), cudaMemcpyDeviceToHost, s));
  BSP_CUDA_TRY(cudaStreamSynchronize(s));
  if (expired) *expired = report[0];
  if (waited_ns) memcpy(waited_ns, &report[2], sizeof(long long));
  return BSP_OK;
}

extern "C" int bsp_linear_status(void* stream) {
  using namespace bsp;
  TcDevice* dev = tc_device();
  if (dev == nullptr) return BSP_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int flag = 0;
  BSP_CUDA_TRY(cudaMemcpyAsync(&flag, dev->status, sizeof(int), cudaMemcpyDeviceToHost, s));
  BSP_CUDA_TRY(cudaStreamSynchronize(s));
  if (flag != 0) {
    BSP_CUDA_TRY(cudaMemsetAsync(dev->status, 0, sizeof(int), s));
    return BSP_ERR_TIMEOUT;
  }
  return BSP_OK;
}
