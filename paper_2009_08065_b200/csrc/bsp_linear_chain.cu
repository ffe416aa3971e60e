// bsp_linear_chain: several pruned linear layers whose inputs are earlier layers' outputs (QKV ->
// attention output -> FFN-up -> FFN-down of an encoder layer), in ONE persistent launch.
// Without attention in between, row-tile m of a layer only needs row-tile m of the layer it reads,
// so the layers need no grid-wide barrier between them.  All output tiles of all layers form one
// list (all tiles of op 0, then op 1, ...; row-tile after row-tile inside an op), and the CTAs take
// tiles from it through a ticket counter: a CTA that is done early simply takes the next tile, so
// the partly filled last wave of one layer is filled with the first tiles of the next, and the
// launch, prologue and drain of every layer but the first and last disappear.
//
// The X producer of a tile first waits until the source rows it reads have been stored: a per
// (op, row-tile) completion counter in global memory, bumped by the epilogue after its TMA stores
// have completed.  A tile only ever waits for tiles with a smaller ticket; every ticket that has
// been handed out belongs to a running CTA that got it without waiting for a larger one, and a CTA
// works through its tiles in the order it took them, so the smallest unfinished tile can always
// proceed: no co-residency of all CTAs is needed.  The dependency wait, like the mbarrier waits,
// has a deadline.
//
// Inside a CTA the pipeline is the one of bsp_linear_tc.cu (X producer, weight producer, MMA
// issuer, two epilogue groups of four warps, two TMEM accumulators, operand stages sized for the
// widest tile); the tile width is chosen per op (256 / 192 / 128 / 64 outputs) and is a run-time
// value here.  The X producer also draws the tickets and hands each one to the other roles through
// a small ring in shared memory (one mbarrier pair per slot).  The weight producer does not wait
// for the source rows, only for free stages, so a tile's first weight tiles are in shared memory
// while its activations are still being written by other SMs.
#include "bsp_tc.cuh"

namespace bsp {
using namespace tc;

int check_linear_args(const void* a, const void* b, const void* c, int n_out, int k_in, int block,
                      const void* X, int tokens, int ldx, int act, const void* Y, int ldy);
int choose_bn(int tokens, int n_out, int sms);

namespace {

constexpr int kMaxBN = 256;
constexpr int kMaxOps = 8;
constexpr int kRing = 4;                     // tickets in flight inside one CTA
constexpr int kChainThreads = kThreads + 32; // 11 warps: X producer, MMA, 8 epilogue, weight producer
using Cfg = TileCfg<kMaxBN>;

struct ChainOp {
  int n_out, k_blocks, act;
  int bn;                // tile width of this op
  int n_tiles;           // output tiles per row-tile (ceil(n_out / bn))
  int tile_begin;        // number of this op's first tile in the list
  int dep;               // op whose output this op reads, or -1 for the chain input
  int dep_need;          // completions of one source row-tile that make it readable
  const uint16_t* bias;
};
struct ChainParams {
  int n_ops, m_tiles, total_tiles, tokens;
  int* done;             // [n_ops][m_tiles] completion counters, then the ticket counter; zeroed before the launch
  int* ticket;
  int* status;
  ChainOp op[kMaxOps];
};
struct ChainMaps {
  CUtensorMap x[kMaxOps], w[kMaxOps], y[kMaxOps];
};

struct TileRef {
  int g, m, n;
};
__device__ __forceinline__ TileRef decode_tile(const ChainParams& P, int t) {
  int g = 0;
  while (g + 1 < P.n_ops && t >= P.op[g + 1].tile_begin) ++g;
  const int local = t - P.op[g].tile_begin;
  const int m = local / P.op[g].n_tiles;
  return TileRef{g, m, local - m * P.op[g].n_tiles};
}

__global__ void __launch_bounds__(kChainThreads, 1)
linear_chain_kernel(const __grid_constant__ ChainMaps M, const __grid_constant__ ChainParams P) {
  constexpr int S = Cfg::kStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  // [S operand stages][4 epilogue staging buffers][bias, bf16, for two tiles][mbarriers, ring, TMEM base]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S * Cfg::kStage + kEpiBytes + 2 * kMaxBN * 2);
  // bars[0..S) full, [S..2S) empty, [2S..2S+2) accumulator full, [2S+2..2S+4) accumulator empty,
  // then kRing "ticket posted" and kRing "ticket read by all" barriers
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 2 * S + 4 + 2 * kRing);
  volatile uint32_t* timed_out = tmem_holder + 1;     // set by a role whose wait expired
  volatile int* s_tile = reinterpret_cast<volatile int*>(tmem_holder + 2);   // [kRing] the ticket of a slot, -1 = no more

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };
  auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * S + a); };
  auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * S + 2 + a); };
  auto posted_bar = [&](int r) { return bar_base + 8u * (2 * S + 4 + r); };
  auto taken_bar = [&](int r) { return bar_base + 8u * (2 * S + 4 + kRing + r); };

  if (threadIdx.x == 0) {
    *timed_out = 0u;
    for (int i = 0; i < P.n_ops; ++i) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&M.x[i])) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&M.w[i])) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&M.y[i])) : "memory");
    }
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 2); mbar_init(empty_bar(s), 1); }   // two producers arm a stage
    for (int a = 0; a < 2; ++a) { mbar_init(acc_full_bar(a), 1); mbar_init(acc_empty_bar(a), 8); }
    for (int r = 0; r < kRing; ++r) { mbar_init(posted_bar(r), 1); mbar_init(taken_bar(r), 3); }   // readers: weights, MMA, epilogue
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

  // Programmatic dependent launch: the set-up above overlapped the previous kernel's tail; everything
  // below reads memory that kernel may have written (the chain input, the weights, the counters).
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // A reader of the ring: waits for slot seq % kRing to be posted for the seq-th time and returns
  // the ticket (-1: no more tiles), or -2 when the wait ran out.
  auto read_ticket = [&](int seq) -> int {
    const int r = seq % kRing;
    if (!mbar_wait(posted_bar(r), static_cast<uint32_t>((seq / kRing) & 1), P.status)) return -2;
    return s_tile[r];
  };

  if (warp == 0 && lane == 0) {
    // ---------------------------------------------------------------- tickets, and TMA producer of the X tiles
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int seq = 0; ok; ++seq) {
      const int r = seq % kRing;
      if (!mbar_wait(taken_bar(r), static_cast<uint32_t>(((seq / kRing) & 1) ^ 1), P.status)) { ok = false; break; }
      int tile = atomicAdd(P.ticket, 1);
      if (tile >= P.total_tiles) tile = -1;
      s_tile[r] = tile;
      mbar_arrive(posted_bar(r));             // (release: the readers' waits acquire the slot's content)
      if (tile < 0) break;
      const TileRef T = decode_tile(P, tile);
      const ChainOp& op = P.op[T.g];
      if (op.dep >= 0) {
        // the rows this tile reads were written by other CTAs' TMA stores
        if (!wait_counter(P.done + op.dep * P.m_tiles + T.m, op.dep_need, P.status)) { ok = false; break; }
        asm volatile("fence.proxy.async;" ::: "memory");   // order the acquire before the async-proxy reads below
      }
      for (int kb = 0; kb < op.k_blocks; ++kb) {
        if (!mbar_wait(empty_bar(stage), phase ^ 1u, P.status)) { ok = false; break; }
        mbar_arrive_expect_tx(full_bar(stage), Cfg::kStageA);
        tma_load_2d(smem_base + stage * Cfg::kStage, &M.x[T.g], kb * kBlockK, T.m * kBlockM, full_bar(stage));
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
    }
    if (!ok) record_timeout(P.status, timed_out);
  } else if (warp == 10 && lane == 0) {
    // ---------------------------------------------------------------- TMA producer of the weight tiles
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int seq = 0; ok; ++seq) {
      const int tile = read_ticket(seq);
      if (tile == -2) { ok = false; break; }
      mbar_arrive(taken_bar(seq % kRing));
      if (tile < 0) break;
      const TileRef T = decode_tile(P, tile);
      const ChainOp& op = P.op[T.g];
      for (int kb = 0; kb < op.k_blocks; ++kb) {
        if (!mbar_wait(empty_bar(stage), phase ^ 1u, P.status)) { ok = false; break; }
        mbar_arrive_expect_tx(full_bar(stage), static_cast<uint32_t>(op.bn) * kBlockK * 2u);
        tma_load_2d(smem_base + stage * Cfg::kStage + Cfg::kStageA, &M.w[T.g], kb * kBlockK, T.n * op.bn, full_bar(stage));
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
    for (int seq = 0; ok; ++seq) {
      const int tile = read_ticket(seq);
      if (tile == -2) { ok = false; break; }
      mbar_arrive(taken_bar(seq % kRing));
      if (tile < 0) break;
      const ChainOp& op = P.op[decode_tile(P, tile).g];
      const uint32_t idesc = instr_desc_bf16(op.bn);
      if (!mbar_wait(acc_empty_bar(acc), acc_phase[acc] ^ 1u, P.status)) { ok = false; break; }
      tcgen05_fence_after();
      const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * kMaxBN);
      for (int kb = 0; kb < op.k_blocks; ++kb) {
        if (!mbar_wait(full_bar(stage), phase, P.status)) { ok = false; break; }
        tcgen05_fence_after();
        const uint32_t a_addr = smem_base + stage * Cfg::kStage;
        const uint32_t b_addr = a_addr + Cfg::kStageA;
#pragma unroll
        for (int k = 0; k < kBlockK / kUmmaK; ++k)
          tcgen05_mma_bf16(d_tmem, smem_desc_sw128(a_addr + k * kUmmaK * 2), smem_desc_sw128(b_addr + k * kUmmaK * 2),
                           idesc, (kb | k) != 0 ? 1u : 0u);
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
    // ---------------------------------------------------------------- epilogue (two groups of four warps)
    const int group = (warp - 2) >> 2;
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int epi_tid = threadIdx.x - 64;
    const bool issuer = (epi_tid & 127) == 0;
    const uint32_t buf0 = smem_base + S * Cfg::kStage + group * 2 * kEpiStage;   // this group's two staging buffers
    uint32_t my_piece = 0;                   // pieces staged by this group so far: selects the buffer
    uint16_t* s_bias = reinterpret_cast<uint16_t*>(smem + S * Cfg::kStage + kEpiBytes);   // [2][256] bf16
    const uint32_t row_off = static_cast<uint32_t>(row) * 64u;
    const uint32_t row_xor = static_cast<uint32_t>((row >> 1) & 3);
    uint32_t acc_phase[2] = {0u, 0u};
    int acc = 0;
    bool ok = true;
    for (int seq = 0; ok; ++seq) {
      // every epilogue thread reads the slot itself; all take the same decision (common vote)
      const int tile = read_ticket(seq);
      if (!epilogue_all_ok(tile != -2)) { ok = false; break; }
      if (tile < 0) {
        if (epi_tid == 0) mbar_arrive(taken_bar(seq % kRing));
        break;
      }
      const TileRef T = decode_tile(P, tile);
      const ChainOp& op = P.op[T.g];
      const int bn = op.bn;
      const int m0 = T.m * kBlockM, n0 = T.n * bn;
      for (int c = epi_tid; c < bn; c += 256)
        s_bias[acc * kMaxBN + c] = (op.bias != nullptr && n0 + c < op.n_out) ? __ldg(op.bias + n0 + c) : static_cast<uint16_t>(0);
      epilogue_sync_all();                   // (every thread has read the slot: it may be reused)
      if (epi_tid == 0) mbar_arrive(taken_bar(seq % kRing));
      if (!epilogue_all_ok(mbar_wait(acc_full_bar(acc), acc_phase[acc], P.status))) { ok = false; break; }
      tcgen05_fence_after();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(acc * kMaxBN);
      const int pieces = (min(bn, op.n_out - n0) + kEpiCols - 1) / kEpiCols;
      bool released = false;
#pragma unroll 1
      for (int pc = group; pc < pieces; pc += 2) {
        const int c0 = pc * kEpiCols;
        const uint32_t buf = buf0 + (my_piece & 1u) * kEpiStage;
        ++my_piece;
        EpiloguePiece piece;
        piece_load(taddr + c0, smem_u32(s_bias + acc * kMaxBN + c0), piece);
        if (issuer) tma_store_wait_read<1>();   // the store issued two pieces ago has read this buffer
        group_sync(group);
        if (pc + 2 >= pieces) {
          tcgen05_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(acc_empty_bar(acc));
          released = true;
        }
        piece_store(piece, op.act, buf + row_off, row_xor);
        fence_async_smem();
        group_sync(group);
        if (issuer) {
          tma_store_2d(&M.y[T.g], n0 + c0, m0, buf);
          tma_store_commit();
        }
      }
      if (!released) {
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty_bar(acc));
      }
      // publish this group's share of the tile: its stores have to be complete (not merely read out
      // of shared memory) before a consumer on another SM may load the rows
      if (issuer) {
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        asm volatile("fence.proxy.async;" ::: "memory");
        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(P.done + T.g * P.m_tiles + T.m) : "memory");
      }
      acc_phase[acc] ^= 1u;
      acc ^= 1;
    }
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

extern "C" int bsp_linear_chain_ws_bytes(int n_ops, int tokens, size_t* bytes) {
  using namespace bsp;
  if (n_ops <= 0 || n_ops > kMaxOps || tokens < 0 || bytes == nullptr) return BSP_ERR_ARG;
  const size_t m_tiles = (static_cast<size_t>(tokens) + kBlockM - 1) / kBlockM;
  *bytes = round_up(sizeof(int) * (n_ops * (m_tiles ? m_tiles : 1) + 1), 256);     // the counters and the ticket
  return BSP_OK;
}

extern "C" int bsp_linear_chain(const bsp_chain_op* ops, int n_ops, const void* X, int tokens, int ldx,
                                void* ws, size_t ws_bytes, void* stream) {
  using namespace bsp;
  if (ops == nullptr || X == nullptr || ws == nullptr) return BSP_ERR_ARG;
  size_t need = 0;
  int st = bsp_linear_chain_ws_bytes(n_ops, tokens, &need);
  if (st != BSP_OK) return st;
  if (!aligned_to(ws, 256) || !aligned_to(X, 16) || ldx % 8) return BSP_ERR_ARG;
  if (ws_bytes < need) return BSP_ERR_WORKSPACE;
  const int m_tiles = (tokens + kBlockM - 1) / kBlockM;
  TcDevice* dev = tc_device();
  if (dev == nullptr) return BSP_ERR_CUDA;

  ChainParams P = {};
  ChainMaps M;
  P.n_ops = n_ops;
  P.m_tiles = m_tiles;
  P.tokens = tokens;
  int tile_begin = 0;
  for (int i = 0; i < n_ops; ++i) {
    const bsp_chain_op& u = ops[i];
    const void* src = X;
    int src_ld = ldx, src_cols = ldx;
    if (u.src >= i) return BSP_ERR_ARG;                        // a source must be an earlier op
    if (u.src >= 0) { src = ops[u.src].Y; src_ld = ops[u.src].ldy; src_cols = ops[u.src].n_out; }
    st = check_linear_args(u.plan, u.plan, u.plan, u.n_out, u.k_in, u.block, src, tokens, src_ld, u.act, u.Y, u.ldy);
    if (st != BSP_OK) return st;
    if (u.src_col < 0 || u.src_col % 8 || u.src_col + u.k_in > src_cols) return BSP_ERR_SHAPE;
    if (!aligned_to(u.plan, 16) || !aligned_to(u.Y, 16) || u.k_in % 8 || u.n_out % 8 || u.ldy % 8 || src_ld % 8)
      return BSP_ERR_UNSUPPORTED;
    if (tokens == 0) continue;
    const int bn = choose_bn(tokens, u.n_out, dev->sms);
    const uint16_t* src_base = static_cast<const uint16_t*>(src) + u.src_col;
    if (!make_map(&M.x[i], src_base, u.k_in, tokens, src_ld, kBlockM)) return BSP_ERR_CUDA;
    if (!make_map(&M.w[i], u.plan, u.k_in, u.n_out, u.k_in, bn)) return BSP_ERR_CUDA;
    if (!make_map(&M.y[i], u.Y, u.n_out, tokens, u.ldy, kBlockM, kEpiCols)) return BSP_ERR_CUDA;
    ChainOp& o = P.op[i];
    o.n_out = u.n_out;
    o.k_blocks = (u.k_in + kBlockK - 1) / kBlockK;
    o.act = u.act;
    o.bn = bn;
    o.n_tiles = (u.n_out + bn - 1) / bn;
    o.tile_begin = tile_begin;
    o.dep = u.src;
    o.dep_need = u.src >= 0 ? 2 * P.op[u.src].n_tiles : 0;   // each tile is published by its two epilogue groups
    o.bias = static_cast<const uint16_t*>(u.bias);
    tile_begin += o.n_tiles * m_tiles;
  }
  if (tokens == 0) return BSP_OK;
  P.total_tiles = tile_begin;

  P.status = dev->status;
  P.done = static_cast<int*>(ws);
  P.ticket = P.done + n_ops * m_tiles;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  BSP_CUDA_TRY(cudaMemsetAsync(ws, 0, need, s));
  if (!dev->attr_set[4]) {
    BSP_CUDA_TRY(cudaFuncSetAttribute(linear_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
    dev->attr_set[4] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(P.total_tiles < dev->sms ? P.total_tiles : dev->sms);
  cfg.blockDim = dim3(kChainThreads);
  cfg.dynamicSmemBytes = Cfg::kSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // the set-up overlaps what precedes in the stream
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  BSP_CUDA_TRY(cudaLaunchKernelEx(&cfg, linear_chain_kernel, M, P));
  return BSP_OK;
}
