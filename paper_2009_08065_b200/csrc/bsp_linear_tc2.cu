// CTA-pair variant of the tensor-core linear kernel (tcgen05 cta_group::2).
//
// The one-CTA kernel streams (128 + BN) x 64 operand elements from L2 per 128 x BN x 64 block of
// multiply-adds, and at BERT shapes it is the L2 -> SM operand traffic, not the tensor pipe, that
// binds (about 9.5 TB/s in aggregate).  Here two CTAs of a cluster share one 256 x 256 output
// tile: each loads its own 128 rows of X and HALF of the 256 weight rows, and one
// tcgen05.mma.cta_group::2 (M = 256) issued by the leader CTA reads both CTAs' shared memory and
// writes rows 0..127 / 128..255 of the accumulator into the two CTAs' tensor memories.  Per CTA
// that is (128 + 128) x 64 elements per block instead of (128 + 256) x 64: one third less
// operand traffic for the same arithmetic.
//
// Roles per CTA: warp 0 lane 0 TMA producer (own A rows, own half of B; completion is counted
// on the leader's mbarrier), warp 1 lane 0 of the LEADER issues the MMAs and commits to both
// CTAs' barriers, warps 2..9 epilogue of the CTA's own 128 rows (as in the one-CTA kernel).
// No TMA multicast is used.  All mbarrier waits are bounded.
#include "bsp_tc.cuh"

namespace bsp {
using namespace tc;

namespace {

constexpr int kPairBN = 256;
constexpr int kPairStageA = kBlockM * kBlockK * 2;         // this CTA's 128 rows of X
constexpr int kPairStageB = (kPairBN / 2) * kBlockK * 2;   // this CTA's 128 of the 256 weight rows
constexpr int kPairStage = kPairStageA + kPairStageB;
constexpr int kPairFixed = 1024 + kEpiBytes + 2 * kPairBN * 2 + 256;
constexpr int kPairStages = (kSmemLimit - kPairFixed) / kPairStage > 8 ? 8 : (kSmemLimit - kPairFixed) / kPairStage;
constexpr int kPairSmemBytes = kPairStages * kPairStage + kPairFixed;
constexpr int kPairTmemCols = 512;

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA load whose completion bytes are counted on an mbarrier that may live in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar_cluster)
      : "memory");
}
__device__ __forceinline__ void tcgen05_commit_pair(uint32_t bar_cluster) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_cluster) : "memory");
}
__device__ __forceinline__ void tcgen05_mma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                      uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
// bf16 x bf16 -> float32, K-major operands, M = 256 (128 rows in each CTA of the pair), N = 256.
constexpr uint32_t kPairIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kPairBN >> 3) << 17) |
                                (static_cast<uint32_t>(256 >> 4) << 24);

struct PairParams {
  int tokens, n_out, k_in, act;
  const uint16_t* bias;
  int* status;
};

__global__ void __launch_bounds__(kThreads, 1)
linear_tc_pair_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                      const __grid_constant__ CUtensorMap map_y, PairParams P) {
  constexpr int S = kPairStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  // [S operand stages][2 epilogue staging buffers][bias, bf16, for two tiles][mbarriers, TMEM base]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S * kPairStage + kEpiBytes + 2 * kPairBN * 2);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 2 * S + 4);
  volatile uint32_t* timed_out = tmem_holder + 1;     // set by a role of this CTA whose wait expired

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0 = leader of the pair
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };                 // used in the leader only
  auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };          // one per CTA
  auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * S + a); };   // one per CTA
  auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * S + 2 + a); };   // used in the leader only

  if (threadIdx.x == 0) {
    *timed_out = 0u;
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_x)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_w)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_y)) : "memory");
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(acc_full_bar(a), 1); mbar_init(acc_empty_bar(a), 16); }   // 8 warps x 2 CTAs
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {   // the same warp in both CTAs, same destination offset
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)),
                 "r"(static_cast<uint32_t>(kPairTmemCols)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tcgen05_fence_before();
  __syncthreads();
  cluster_sync_all();          // both CTAs' barriers exist before anything signals across the pair
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const int m_tiles = (P.tokens + 255) / 256;
  const int n_tiles = (P.n_out + kPairBN - 1) / kPairBN;
  const int total_tiles = m_tiles * n_tiles;
  const int k_blocks = (P.k_in + kBlockK - 1) / kBlockK;

  if (warp == 0 && lane == 0) {
    // ---------------------------------------------------------------- TMA producer (both CTAs)
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
      const int m0 = (tile / n_tiles) * 256 + static_cast<int>(rank) * kBlockM;
      const int w0 = (tile % n_tiles) * kPairBN + static_cast<int>(rank) * (kPairBN / 2);
      for (int kb = 0; kb < k_blocks; ++kb) {
        if (!mbar_wait(empty_bar(stage), phase ^ 1u, P.status)) { ok = false; break; }
        const uint32_t a_dst = smem_base + stage * kPairStage;
        const uint32_t b_dst = a_dst + kPairStageA;
        const uint32_t leader_full = map_to_cta(full_bar(stage), 0);
        if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), 2 * kPairStage);   // both CTAs' bytes
        tma_load_2d_pair(a_dst, &map_x, kb * kBlockK, m0, leader_full);
        tma_load_2d_pair(b_dst, &map_w, kb * kBlockK, w0, leader_full);
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
    }
    if (!ok) record_timeout(P.status, timed_out);
  } else if (warp == 1 && lane == 0 && rank == 0) {
    // ---------------------------------------------------------------- MMA issuer (leader CTA only)
    int stage = 0;
    uint32_t phase = 0;
    uint32_t acc_phase[2] = {0u, 0u};
    int acc = 0;
    bool ok = true;
    for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
      if (!mbar_wait(acc_empty_bar(acc), acc_phase[acc] ^ 1u, P.status)) { ok = false; break; }
      tcgen05_fence_after();
      const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * kPairBN);
      for (int kb = 0; kb < k_blocks; ++kb) {
        if (!mbar_wait(full_bar(stage), phase, P.status)) { ok = false; break; }
        tcgen05_fence_after();
        const uint32_t a_addr = smem_base + stage * kPairStage;
        const uint32_t b_addr = a_addr + kPairStageA;
#pragma unroll
        for (int k = 0; k < kBlockK / kUmmaK; ++k)
          tcgen05_mma_bf16_pair(d_tmem, smem_desc_sw128(a_addr + k * kUmmaK * 2), smem_desc_sw128(b_addr + k * kUmmaK * 2),
                                kPairIdesc, (kb | k) != 0 ? 1u : 0u);
        // the stage is free in both CTAs once these MMAs have read it
        tcgen05_commit_pair(empty_bar(stage));
        tcgen05_commit_pair(map_to_cta(empty_bar(stage), 1));
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
      if (!ok) break;
      tcgen05_commit_pair(acc_full_bar(acc));
      tcgen05_commit_pair(map_to_cta(acc_full_bar(acc), 1));
      acc_phase[acc] ^= 1u;
      acc ^= 1;
    }
    if (!ok) record_timeout(P.status, timed_out);
  } else if (warp >= 2) {
    // ---------------------------------------------------------------- epilogue of this CTA's 128 rows
    const int group = (warp - 2) >> 2;
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int epi_tid = threadIdx.x - 64;
    const bool issuer = (epi_tid & 127) == 0;
    const uint32_t buf0 = smem_base + S * kPairStage + group * 2 * kEpiStage;   // this group's two staging buffers
    uint32_t my_piece = 0;                   // pieces staged by this group so far: selects the buffer
    uint16_t* s_bias = reinterpret_cast<uint16_t*>(smem + S * kPairStage + kEpiBytes);
    const uint32_t row_off = static_cast<uint32_t>(row) * 64u;
    const uint32_t row_xor = static_cast<uint32_t>((row >> 1) & 3);
    uint32_t acc_phase[2] = {0u, 0u};
    int acc = 0;
    bool ok = true;
    for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
      const int m0 = (tile / n_tiles) * 256 + static_cast<int>(rank) * kBlockM, n0 = (tile % n_tiles) * kPairBN;
      for (int c = epi_tid; c < kPairBN; c += 256)
        s_bias[acc * kPairBN + c] = (P.bias != nullptr && n0 + c < P.n_out) ? __ldg(P.bias + n0 + c) : static_cast<uint16_t>(0);
      epilogue_sync_all();
      // all 256 threads take the same decision, so nobody is left alone at a named barrier below
      if (!epilogue_all_ok(mbar_wait(acc_full_bar(acc), acc_phase[acc], P.status))) { ok = false; break; }
      tcgen05_fence_after();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(acc * kPairBN);
      const uint32_t leader_acc_empty = map_to_cta(acc_empty_bar(acc), 0);
      const int pieces = (min(kPairBN, P.n_out - n0) + kEpiCols - 1) / kEpiCols;
      bool released = false;
#pragma unroll 1
      for (int pc = group; pc < pieces; pc += 2) {
        const int c0 = pc * kEpiCols;
        const uint32_t buf = buf0 + (my_piece & 1u) * kEpiStage;
        ++my_piece;
        if (issuer) tma_store_wait_read<1>();   // the store issued two pieces ago has read this buffer
        group_sync(group);
        EpiloguePiece piece;
        piece_load(taddr + c0, smem_u32(s_bias + acc * kPairBN + c0), piece);
        if (pc + 2 >= pieces) {              // this warp's last read of the accumulator
          tcgen05_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(leader_acc_empty);
          released = true;
        }
        piece_store(piece, P.act, buf + row_off, row_xor);
        fence_async_smem();
        group_sync(group);
        if (issuer) {
          tma_store_2d(&map_y, n0 + c0, m0, buf);
          tma_store_commit();
        }
      }
      if (!released) {
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(leader_acc_empty);
      }
      acc_phase[acc] ^= 1u;
      acc ^= 1;
    }
    if (issuer) tma_store_wait_read<0>();
    if (!ok && lane == 0) record_timeout(P.status, timed_out);
  }

  tcgen05_fence_before();
  __syncthreads();
  quiet_period(timed_out);
  cluster_sync_all();          // neither CTA leaves while the other may still touch its memory or barriers
  if (warp == 1) {
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(static_cast<uint32_t>(kPairTmemCols)) : "memory");
  }
}

}  // namespace

// Launch of the CTA-pair kernel (arguments already validated by the caller).
int launch_tc_pair(TcDevice* dev, const void* plan, const void* X, void* Y, int tokens, int n_out, int k_in, int act,
                   const void* bias, int ldx, int ldy, cudaStream_t s) {
  CUtensorMap map_x, map_w, map_y;
  if (!make_map(&map_x, X, k_in, tokens, ldx, kBlockM)) return BSP_ERR_CUDA;
  if (!make_map(&map_w, plan, k_in, n_out, k_in, kPairBN / 2)) return BSP_ERR_CUDA;
  if (!make_map(&map_y, Y, n_out, tokens, ldy, kBlockM, kEpiCols)) return BSP_ERR_CUDA;
  if (!dev->attr_set[5]) {
    BSP_CUDA_TRY(cudaFuncSetAttribute(linear_tc_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmemBytes));
    dev->attr_set[5] = true;
  }
  PairParams P{tokens, n_out, k_in, act, static_cast<const uint16_t*>(bias), dev->status};
  const int tiles = ((tokens + 255) / 256) * ((n_out + kPairBN - 1) / kPairBN);
  const int pairs = tiles < dev->sms / 2 ? tiles : dev->sms / 2;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kPairSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  BSP_CUDA_TRY(cudaLaunchKernelEx(&cfg, linear_tc_pair_kernel, map_x, map_w, map_y, P));
  return BSP_OK;
}

}  // namespace bsp
