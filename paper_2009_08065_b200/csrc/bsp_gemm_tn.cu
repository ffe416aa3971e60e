// bsp_linear_backward_weight: the weight gradient of the masked layer that Algorithm 2 retrains
// (W = W * Mask):  dW = (dY^T X) * Mask,  dY [tokens, n_out], X [tokens, k_in], dW [n_out, k_in].
//
// The contraction runs over tokens, the slow dimension of both operands, so the tensor-core tiles
// are "MN-major": a pipeline stage holds 64 token rows of dY (128 output-row elements wide) and of
// X (256 columns wide), each loaded as boxes of 64 elements x 64 token rows with the 128-byte
// swizzle; in shared memory that is a stack of 1024-byte atoms (8 token rows x 64 elements), 8 KB
// from one 64-element column group to the next, which is what the MN-major form of the tcgen05
// shared-memory descriptor describes (leading byte offset = distance between 64-element groups,
// stride byte offset = distance between 8-row groups).  Everything else (persistent CTAs, TMA
// producers, one MMA-issuing thread, two TMEM accumulators, two epilogue groups, TMA stores,
// bounded waits) is the pipeline of bsp_linear_tc.cu with a 128 x 256 output tile.
// The mask is applied afterwards by the mask kernel (pruned groups of dW are written as zero).
#include "bsp_tc.cuh"

namespace bsp {
using namespace tc;

namespace {

constexpr int kTnBN = 256;
constexpr int kTnThreads = kThreads + 32;          // producer A, MMA, 8 epilogue warps, producer B
using Cfg = TileCfg<kTnBN>;
constexpr int kAtomGroup = 64 * kBlockK * 2;       // 64 elements x 64 token rows = 8 KB

// MN-major operand tile with the 128-byte swizzle: 8-row atoms 1024 bytes apart along the
// contraction, 64-element groups 8 KB apart along M / N.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3ffff) >> 4);
  d |= static_cast<uint64_t>(kAtomGroup >> 4) << 16;            // leading byte offset / 16
  d |= static_cast<uint64_t>(1024 >> 4) << 32;                   // stride byte offset / 16
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
// bf16 x bf16 -> float32, both operands MN-major (bits 15 and 16), M = 128, N = 256.
constexpr uint32_t kTnIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) |
                              (static_cast<uint32_t>(kTnBN >> 3) << 17) | (static_cast<uint32_t>(kBlockM >> 4) << 24);

struct TnParams {
  int tokens, n_out, k_in;
  int* status;
};

__global__ void __launch_bounds__(kTnThreads, 1)
gemm_tn_kernel(const __grid_constant__ CUtensorMap map_dy, const __grid_constant__ CUtensorMap map_x,
               const __grid_constant__ CUtensorMap map_dw, TnParams P) {
  constexpr int S = Cfg::kStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  uint16_t* s_zero = reinterpret_cast<uint16_t*>(smem + S * Cfg::kStage + kEpiBytes);       // zero "bias"
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S * Cfg::kStage + kEpiBytes + 2 * kTnBN * 2);
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
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 2); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(acc_full_bar(a), 1); mbar_init(acc_empty_bar(a), 8); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  for (int c = threadIdx.x; c < 2 * kTnBN; c += blockDim.x) s_zero[c] = 0;
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)),
                 "r"(static_cast<uint32_t>(Cfg::kTmemCols)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // output tile (mt, nt): rows [128 mt, +128) of dW (output features), columns [256 nt, +256) (input features)
  const int m_tiles = (P.n_out + kBlockM - 1) / kBlockM;
  const int n_tiles = (P.k_in + kTnBN - 1) / kTnBN;
  const int total_tiles = m_tiles * n_tiles;
  const int k_blocks = (P.tokens + kBlockK - 1) / kBlockK;

  if (warp == 0 && lane == 0) {
    // ---------------------------------------------------------------- TMA producer of the dY tiles
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int m0 = (tile / n_tiles) * kBlockM;
      for (int kb = 0; kb < k_blocks; ++kb) {
        if (!mbar_wait(empty_bar(stage), phase ^ 1u, P.status)) { ok = false; break; }
        const uint32_t a_dst = smem_base + stage * Cfg::kStage;
        mbar_arrive_expect_tx(full_bar(stage), Cfg::kStageA);
#pragma unroll
        for (int g = 0; g < kBlockM / 64; ++g)
          tma_load_2d(a_dst + g * kAtomGroup, &map_dy, m0 + 64 * g, kb * kBlockK, full_bar(stage));
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
    }
    if (!ok) record_timeout(P.status, timed_out);
  } else if (warp == 10 && lane == 0) {
    // ---------------------------------------------------------------- TMA producer of the X tiles
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int n0 = (tile % n_tiles) * kTnBN;
      for (int kb = 0; kb < k_blocks; ++kb) {
        if (!mbar_wait(empty_bar(stage), phase ^ 1u, P.status)) { ok = false; break; }
        const uint32_t b_dst = smem_base + stage * Cfg::kStage + Cfg::kStageA;
        mbar_arrive_expect_tx(full_bar(stage), Cfg::kStageB);
#pragma unroll
        for (int g = 0; g < kTnBN / 64; ++g)
          tma_load_2d(b_dst + g * kAtomGroup, &map_x, n0 + 64 * g, kb * kBlockK, full_bar(stage));
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
    }
    if (!ok) record_timeout(P.status, timed_out);
  } else if (warp == 1 && lane == 0) {
    // ---------------------------------------------------------------- MMA issuer
    int stage = 0;
    uint32_t phase = 0;
    uint32_t acc_phase[2] = {0u, 0u};
    int acc = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      if (!mbar_wait(acc_empty_bar(acc), acc_phase[acc] ^ 1u, P.status)) { ok = false; break; }
      tcgen05_fence_after();
      const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * kTnBN);
      for (int kb = 0; kb < k_blocks; ++kb) {
        if (!mbar_wait(full_bar(stage), phase, P.status)) { ok = false; break; }
        tcgen05_fence_after();
        const uint32_t a_addr = smem_base + stage * Cfg::kStage;
        const uint32_t b_addr = a_addr + Cfg::kStageA;
#pragma unroll
        for (int k = 0; k < kBlockK / kUmmaK; ++k)     // 16 token rows = two 8-row atoms = 2048 bytes per step
          tcgen05_mma_bf16(d_tmem, smem_desc_mn_sw128(a_addr + k * 2048), smem_desc_mn_sw128(b_addr + k * 2048), kTnIdesc,
                           (kb | k) != 0 ? 1u : 0u);
        tcgen05_commit(empty_bar(stage));
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
      if (!ok) break;
      tcgen05_commit(acc_full_bar(acc));
      acc_phase[acc] ^= 1u;
      acc ^= 1;
    }
    if (!ok) record_timeout(P.status, timed_out);
  } else if (warp >= 2 && warp < 10) {
    // ---------------------------------------------------------------- epilogue (as in bsp_linear_tc.cu, no bias)
    const int group = (warp - 2) >> 2;
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int epi_tid = threadIdx.x - 64;
    const bool issuer = (epi_tid & 127) == 0;
    const uint32_t buf0 = smem_base + S * Cfg::kStage + group * 2 * kEpiStage;
    uint32_t my_piece = 0;
    const uint32_t row_off = static_cast<uint32_t>(row) * 64u;
    const uint32_t row_xor = static_cast<uint32_t>((row >> 1) & 3);
    uint32_t acc_phase[2] = {0u, 0u};
    int acc = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int m0 = (tile / n_tiles) * kBlockM, n0 = (tile % n_tiles) * kTnBN;
      // all 256 threads take the same decision, so nobody is left alone at a named barrier below
      if (!epilogue_all_ok(mbar_wait(acc_full_bar(acc), acc_phase[acc], P.status))) { ok = false; break; }
      tcgen05_fence_after();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(acc * kTnBN);
      const int pieces = (min(kTnBN, P.k_in - n0) + kEpiCols - 1) / kEpiCols;
      bool released = false;
#pragma unroll 1
      for (int pc = group; pc < pieces; pc += 2) {
        const int c0 = pc * kEpiCols;
        const uint32_t buf = buf0 + (my_piece & 1u) * kEpiStage;
        ++my_piece;
        if (issuer) tma_store_wait_read<1>();
        group_sync(group);
        EpiloguePiece piece;
        piece_load(taddr + c0, smem_u32(s_zero), piece);
        if (pc + 2 >= pieces) {
          tcgen05_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(acc_empty_bar(acc));
          released = true;
        }
        piece_store(piece, BSP_ACT_NONE, buf + row_off, row_xor);
        fence_async_smem();
        group_sync(group);
        if (issuer) {
          tma_store_2d(&map_dw, n0 + c0, m0, buf);
          tma_store_commit();
        }
      }
      if (!released) {
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty_bar(acc));
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
  if (warp == 1) {
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(static_cast<uint32_t>(Cfg::kTmemCols)) : "memory");
  }
}

}  // namespace
}  // namespace bsp

extern "C" int bsp_linear_backward_weight(const void* dY, int ldy, const void* X, int ldx, int tokens, int n_out,
                                          int k_in, int block, const uint8_t* keep, void* dW, int lddw, void* stream) {
  using namespace bsp;
  if (dY == nullptr || X == nullptr || dW == nullptr) return BSP_ERR_ARG;
  if (tokens <= 0 || n_out <= 0 || k_in <= 0 || block <= 0) return BSP_ERR_ARG;
  if (n_out % block) return BSP_ERR_SHAPE;
  if (ldy < n_out || ldx < k_in || lddw < k_in) return BSP_ERR_SHAPE;
  if (!aligned_to(dY, 16) || !aligned_to(X, 16) || !aligned_to(dW, 16) || ldy % 8 || ldx % 8 || lddw % 8 || n_out % 8 ||
      k_in % 8)
    return BSP_ERR_UNSUPPORTED;
  TcDevice* dev = tc_device();
  if (dev == nullptr) return BSP_ERR_CUDA;
  // operands as [token rows, features]: inner dimension = features, boxes of 64 features x 64 token rows
  CUtensorMap map_dy, map_x, map_dw;
  if (!make_map(&map_dy, dY, n_out, tokens, ldy, kBlockK)) return BSP_ERR_CUDA;
  if (!make_map(&map_x, X, k_in, tokens, ldx, kBlockK)) return BSP_ERR_CUDA;
  if (!make_map(&map_dw, dW, k_in, n_out, lddw, kBlockM, kEpiCols)) return BSP_ERR_CUDA;
  if (!dev->attr_set[6]) {
    BSP_CUDA_TRY(cudaFuncSetAttribute(gemm_tn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
    dev->attr_set[6] = true;
  }
  TnParams P{tokens, n_out, k_in, dev->status};
  const int tiles = ((n_out + kBlockM - 1) / kBlockM) * ((k_in + kTnBN - 1) / kTnBN);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(tiles < dev->sms ? tiles : dev->sms);
  cfg.blockDim = dim3(kTnThreads);
  cfg.dynamicSmemBytes = Cfg::kSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  BSP_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_tn_kernel, map_dy, map_x, map_dw, P));
  if (keep != nullptr) return bsp_apply_mask(dW, n_out, k_in, lddw, block, BSP_ORIENT_C, keep, stream);
  return BSP_OK;
}
