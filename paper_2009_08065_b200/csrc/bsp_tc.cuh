// Building blocks of the tensor-core kernels: tile constants, PTX wrappers (mbarrier, TMA, tcgen05,
// TMEM), shared-memory / instruction descriptors, the epilogue math, and the host-side tensor-map
// encoder.  Shared by bsp_linear_tc.cu (one linear per launch) and bsp_linear_chain.cu (a chain
// of linears in one persistent launch).
#pragma once

#include <cuda.h>
#include <math.h>

#include "bsp_common.cuh"

namespace bsp {
namespace tc {

constexpr int kBlockM = 128;      // tokens per tile (TMEM lanes)
constexpr int kBlockK = 64;       // bf16 elements per pipeline stage row = 128 bytes = one swizzle row
constexpr int kUmmaK = 16;        // K of one tcgen05.mma for 16-bit inputs
constexpr int kThreads = 320;     // 10 warps: producer, mma, 2 x 4 epilogue
constexpr int kSmemLimit = 232448;              // 227 KB of dynamic shared memory per CTA
constexpr int kEpiCols = 32;                    // columns per epilogue piece = one 64-byte swizzle row of bf16
constexpr int kEpiStage = kBlockM * kEpiCols * 2;     // one staging buffer: 128 rows x 64 bytes
constexpr int kEpiBuffers = 4;                  // two per epilogue group, so a store can drain while the next piece is staged
constexpr int kEpiBytes = kEpiBuffers * kEpiStage;
constexpr unsigned long long kDefaultWaitLimitNs = 2000000000ull;  // 2 s per wait unless bsp_set_wait_limit_ms says otherwise
constexpr unsigned long long kQuietNs = 1000000ull;         // 1 ms for operations in flight after a wait gave up


// Shared-memory plan of a CTA for an output tile 128 x BN: operand stages, two epilogue staging
// buffers, the bias of two tiles (bf16), the mbarriers.
template <int BN>
struct TileCfg {
  static constexpr int kStageA = kBlockM * kBlockK * 2;
  static constexpr int kStageB = BN * kBlockK * 2;
  static constexpr int kStage = kStageA + kStageB;
  static constexpr int kFixed = 1024 /*alignment slack*/ + kEpiBytes + 2 * BN * 2 /*bias, two tiles*/ + 256 /*barriers*/;
  static constexpr int kStages = ((kSmemLimit - kFixed) / kStage) > 8 ? 8 : ((kSmemLimit - kFixed) / kStage);
  static constexpr int kTmemCols = 2 * BN <= 32 ? 32 : 2 * BN <= 64 ? 64 : 2 * BN <= 128 ? 128 : 2 * BN <= 256 ? 256 : 512;
  static constexpr int kSmemBytes = kStages * kStage + kFixed;
};

#ifdef __CUDACC__
// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// The status area of a device is four 32-bit words: [0] the status code that kernels set when a
// bounded wait expires, [1] unused, [2..3] the limit of one wait in nanoseconds (64 bits).
__device__ __forceinline__ unsigned long long wait_limit_ns(const int* status) {
  return *reinterpret_cast<const volatile unsigned long long*>(status + 2);
}
// Bounded wait: false when the deadline passed (the caller records the failure and bails out).
// The limit is read only once the first probe has failed.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long limit = wait_limit_ns(status);
  const unsigned long long start = global_timer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (global_timer_ns() - start > limit) return false;
  }
}
// The same wait for many threads at once (a whole CTA waiting for its bulk copies): each probe lets
// the hardware suspend the thread for up to `kSuspendNs` or until the phase completes, so the
// waiting warps leave the issue slots to the CTAs that share the SM instead of polling.
constexpr uint32_t kSuspendNs = 4000u;
__device__ __forceinline__ bool mbar_try_wait_suspend(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(kSuspendNs)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_suspended(uint32_t bar, uint32_t parity, const int* status) {
  if (mbar_try_wait_suspend(bar, parity)) return true;
  const unsigned long long limit = wait_limit_ns(status);
  const unsigned long long start = global_timer_ns();
  for (;;) {
    if (mbar_try_wait_suspend(bar, parity)) return true;
    if (global_timer_ns() - start > limit) return false;
  }
}
// Bounded wait until *counter >= need (acquire at GPU scope): a counter in global memory that
// other CTAs of the same launch bump.
__device__ __forceinline__ bool wait_counter(const int* counter, int need, const int* status) {
  const unsigned long long limit = wait_limit_ns(status);
  const unsigned long long start = global_timer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) {
      int v;
      asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
      if (v >= need) return true;
    }
    if (global_timer_ns() - start > limit) return false;
  }
}
// A role whose wait expired: the device-wide status word for the host, and this CTA's own flag so that
// the CTA holds on to its shared and tensor memory for a while before it exits (see quiet_period).
__device__ __forceinline__ void record_timeout(int* status, volatile uint32_t* cta_flag) {
  atomicExch(status, BSP_ERR_TIMEOUT);
  *cta_flag = 1u;
}
// After a wait gave up, copies and tensor-core operations that were already issued may still be
// writing this CTA's shared or tensor memory; they complete within microseconds once their data
// arrives.  The CTA waits a fixed millisecond before it gives that memory back.  Call after the
// block-wide barrier that follows the role loops; every thread takes part.
__device__ __forceinline__ void quiet_period(const volatile uint32_t* cta_flag) {
  if (*cta_flag != 0u) {
    const unsigned long long start = global_timer_ns();
    while (global_timer_ns() - start < kQuietNs) __nanosleep(2000);
  }
  __syncthreads();
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tcgen05_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_load_32cols(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int x, int y, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(src)
               : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void tma_store_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// Named barriers of the epilogue (barrier 0 is __syncthreads): 1 + g among the 128 threads of
// epilogue group g, 3 among all 256 epilogue threads.
__device__ __forceinline__ void group_sync(int g) { asm volatile("bar.sync %0, 128;" ::"r"(1 + g) : "memory"); }
__device__ __forceinline__ void epilogue_sync_all() { asm volatile("bar.sync 3, 256;" ::: "memory"); }
// The 256 epilogue threads agree on whether all of their waits succeeded (named barrier 4 with an AND
// reduction): either every one of them goes on to the named barriers of the tile, or none does.
__device__ __forceinline__ bool epilogue_all_ok(bool ok) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 p, %1, 0;\n\t"
      "barrier.cta.red.and.pred q, 4, 256, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r)
      : "r"(ok ? 1u : 0u)
      : "memory");
  return r != 0u;
}
// Shared-memory accesses of the epilogue as volatile asm WITHOUT a memory clobber: they keep their
// order among themselves and with the fences and barriers around them (all volatile asm), but do
// not stop the compiler from hoisting the bias loads of a whole piece ahead of its stores.
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d));
}
__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void tmem_load_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 tile stored as 128-byte swizzled rows
// (what a TMA load with the 128-byte swizzle mode writes): 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3ffff) >> 4);        // start address / 16
  d |= static_cast<uint64_t>(1) << 16;                           // leading byte offset / 16 (unused with swizzle)
  d |= static_cast<uint64_t>(1024 >> 4) << 32;                   // stride byte offset / 16
  d |= static_cast<uint64_t>(1) << 46;                           // descriptor version of this architecture
  d |= static_cast<uint64_t>(2) << 61;                           // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> float32, both operands K-major, M = 128, N = BN.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(kBlockM >> 4) << 24);
}

// GELU(x) = x * Phi(x), Phi the standard normal distribution function (the erf form, 0.5 (1 + erf(x / sqrt 2))).
// The lower tail is evaluated as Phi(-a) = 2^(-P(a)), a = min(|x|, 6), with P a degree-5 polynomial
// fitted by weighted least squares to -log2 Phi(-a) on [0, 6]; the largest absolute error of Phi in
// float32 is 3.2e-7 (below 1e-9 beyond a = 6), so x Phi(x) is off by at most 2e-6 in absolute terms,
// far under the bf16 rounding of the output except deep in the lower tail.  One
// special-function operation (ex2) per element, no branch, no select: with q = Phi(-|x|),
// x Phi(x) = max(x, 0) - |x| q for either sign of x.
__device__ __forceinline__ float gelu_erf(float x) {
  const float a = fminf(fabsf(x), 6.0f);
  float p = fmaf(-0.000518865308f, a, 0.00738722592f);
  p = fmaf(p, a, -0.0525380379f);
  p = fmaf(p, a, -0.459276694f);
  p = fmaf(p, a, -1.15108313f);
  p = fmaf(p, a, -1.00000084f);
  float q;                                   // q = Phi(-|x|); the argument is in [-28, -1], far from any special case
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(q) : "f"(p));
  // x Phi(x) = max(x, 0) - |x| q for either sign of x: no compare, no select, and no cancellation
  // in the lower tail (for x < 0 the result is -|x| q, rounded once)
  return fmaf(-fabsf(x), q, fmaxf(x, 0.0f));
}

// Two float32 values as one 64-bit register pair, and the packed float32 FMA of this architecture
// (fma.rn.f32x2: two independent correctly rounded FMAs in one instruction, so a result is bit for
// bit what fmaf gives).
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
// gelu_erf for two values at once: the same operations in the same order per value, with the five
// polynomial steps issued as packed FMAs (the epilogue of a GELU layer is bound by instruction issue).
__device__ __forceinline__ void gelu_erf_pair(float& x0, float& x1) {
  const unsigned long long a = pack_f32x2(fminf(fabsf(x0), 6.0f), fminf(fabsf(x1), 6.0f));
  unsigned long long p = fma_f32x2(pack_f32x2(-0.000518865308f, -0.000518865308f), a, pack_f32x2(0.00738722592f, 0.00738722592f));
  p = fma_f32x2(p, a, pack_f32x2(-0.0525380379f, -0.0525380379f));
  p = fma_f32x2(p, a, pack_f32x2(-0.459276694f, -0.459276694f));
  p = fma_f32x2(p, a, pack_f32x2(-1.15108313f, -1.15108313f));
  p = fma_f32x2(p, a, pack_f32x2(-1.00000084f, -1.00000084f));
  float p0, p1, q0, q1;
  unpack_f32x2(p, p0, p1);
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(q0) : "f"(p0));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(q1) : "f"(p1));
  x0 = fmaf(-fabsf(x0), q0, fmaxf(x0, 0.0f));
  x1 = fmaf(-fabsf(x1), q1, fmaxf(x1, 0.0f));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));   // upper half <- first source
  return r;
}

// One 32-column piece of a thread's accumulator row, with the bias of those columns.
struct EpiloguePiece {
  uint32_t v[32];            // float32 accumulators as bits
  uint4 bias[4];             // 32 bf16 values
};
// Issues the TMEM load and, while it is in flight, the four shared-memory loads of the bias;
// returns once the accumulator values are in registers.  Shared memory is also being written by
// TMA and read by the tensor core all the time, so a shared load takes on the order of 150 cycles
// here: the loads must be in flight together, not one per use.
__device__ __forceinline__ void piece_load(uint32_t taddr, uint32_t bias_smem, EpiloguePiece& p) {
  tmem_load_32cols(taddr, p.v);
#pragma unroll
  for (int j = 0; j < 4; ++j) p.bias[j] = ld_shared_v4(bias_smem + 16u * j);
  tmem_load_wait();
}
// bias + optional GELU + bf16 rounding, into this thread's 64-byte row of a staging buffer laid out
// as a TMA store with the 64-byte swizzle expects it (16-byte chunk c of row r at chunk c ^ ((r >> 1) & 3)).
__device__ __forceinline__ void piece_store(const EpiloguePiece& p, int act, uint32_t dst_row, uint32_t row_xor) {
#pragma unroll
  for (int j = 0; j < 4; ++j) {        // 8 outputs -> one 16-byte chunk
    const uint32_t* v = &p.v[j * 8];
    const uint32_t bw[4] = {p.bias[j].x, p.bias[j].y, p.bias[j].z, p.bias[j].w};
    float f[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(v[2 * i]) + __uint_as_float(bw[i] << 16);
      f[2 * i + 1] = __uint_as_float(v[2 * i + 1]) + __uint_as_float(bw[i] & 0xffff0000u);
    }
    if (act == BSP_ACT_GELU) {
#pragma unroll
      for (int i = 0; i < 8; i += 2) gelu_erf_pair(f[i], f[i + 1]);
    }
    st_shared_v4(dst_row + ((static_cast<uint32_t>(j) ^ row_xor) << 4), pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]),
                 pack_bf16x2(f[4], f[5]), pack_bf16x2(f[6], f[7]));
  }
}
// The same piece for a TRANSPOSED output [n_out, tokens]: the staging buffer is 32 output rows of 128
// tokens (256 bytes each, no swizzle); this thread's token is column `row`, so the 32 lanes of a warp
// write 64 contiguous bytes per output row.
__device__ __forceinline__ void piece_store_transposed(const EpiloguePiece& p, int act, uint32_t buf, int row) {
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint32_t* v = &p.v[j * 8];
    const uint32_t bw[4] = {p.bias[j].x, p.bias[j].y, p.bias[j].z, p.bias[j].w};
    float f[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(v[2 * i]) + __uint_as_float(bw[i] << 16);
      f[2 * i + 1] = __uint_as_float(v[2 * i + 1]) + __uint_as_float(bw[i] & 0xffff0000u);
    }
    if (act == BSP_ACT_GELU) {
#pragma unroll
      for (int i = 0; i < 8; i += 2) gelu_erf_pair(f[i], f[i + 1]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t w = pack_bf16x2(f[2 * i], f[2 * i + 1]);
      const uint32_t a = buf + static_cast<uint32_t>((j * 8 + 2 * i) * 256 + row * 2);
      asm volatile("st.shared.b16 [%0], %1;" ::"r"(a), "h"(static_cast<uint16_t>(w & 0xffffu)));
      asm volatile("st.shared.b16 [%0], %1;" ::"r"(a + 256u), "h"(static_cast<uint16_t>(w >> 16)));
    }
  }
}
#endif  // __CUDACC__

// ------------------------------------------------------------------------------------------
// host side: tensor maps
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// 2-D bf16 tensor [outer, inner] row-major with leading dimension ld; box [box_outer, box_inner]:
// 64 columns with the 128-byte swizzle (operand tiles) or 32 columns with the 64-byte swizzle
// (epilogue pieces); out-of-range elements read as zero and are not written.
// A box of 128 columns is stored without a swizzle (the staging buffer of a transposed output piece).
inline bool make_map(CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer, uint64_t ld, uint32_t box_outer,
                     uint32_t box_inner = 64, CUtensorMapL2promotion promote = CU_TENSOR_MAP_L2_PROMOTION_L2_256B) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {inner, outer};
  const cuuint64_t strides[1] = {ld * 2};
  const cuuint32_t box[2] = {box_inner, box_outer};
  const cuuint32_t elem[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
            CU_TENSOR_MAP_INTERLEAVE_NONE,
            box_inner == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : box_inner == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE, promote,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


}  // namespace tc

// Per-device facts the launchers need: SM count and the device address of the status word that
// a kernel sets when one of its bounded waits expires.  Null on failure.
struct TcDevice {
  int sms = 0;
  int* status = nullptr;
  bool attr_set[8] = {false, false, false, false, false, false, false, false};
};
TcDevice* tc_device();

}  // namespace bsp
