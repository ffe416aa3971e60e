// bsp_linear_route / bsp_linear_run / bsp_linear_tune: one front door for the pruned linear layer.
//
// The library has two ways to run Y = act(X (W * Mask)^T + b): the zero-expanded route
// (bsp_linear_planned_ex: dense tcgen05 tiles over W with zeros in the pruned places; executes
// 2 T N K flops whatever the compression) and the gathering route (bsp_linear_gathered_ex: only the
// kept columns are fetched and multiplied; its time per 64 kept columns does not depend on the
// block height).  Which is faster depends on the block height, the compression, the shape and the
// activation.  The caller describes what it has (which layouts of the weights, which layouts of the
// activations, which layout it wants out) and either names a route, lets a cost estimate fitted to
// measurements choose, or has both timed on the spot.
#include <cuda_runtime.h>

#include "bsp_common.cuh"

namespace bsp {
namespace {

bool gather_block(int block) { return block == 16 || block == 32 || block == 64 || block == 128; }

bool can_zero_expanded(const bsp_linear_call& c) { return c.plan != nullptr && c.X != nullptr; }
bool can_gathered(const bsp_linear_call& c) { return c.gplan != nullptr && c.XT != nullptr && gather_block(c.block); }

int check_call(const bsp_linear_call* c) {
  if (c == nullptr) return BSP_ERR_ARG;
  if (c->n_out <= 0 || c->k_in <= 0 || c->block <= 0 || c->tokens < 0) return BSP_ERR_ARG;
  if (c->n_out % c->block) return BSP_ERR_SHAPE;
  if ((c->Y == nullptr) == (c->YT == nullptr)) return BSP_ERR_ARG;          // exactly one output layout
  if (c->X == nullptr && c->XT == nullptr) return BSP_ERR_ARG;
  if (c->plan == nullptr && c->gplan == nullptr) return BSP_ERR_ARG;
  return BSP_OK;
}

// Estimated microseconds of the two routes on `sms` SMs.  Zero-expanded: the dense product at the
// rate the kernel sustains (lower with GELU in the epilogue).  Gathering: every CTA works through
// (token tile) x (row-block) units; a stage of 64 kept columns costs 0.62 us (the TMA row gather is the
// bound, whatever the block height) and every row-block 0.45 us more (accumulator hand-over).
void estimate_us(const bsp_linear_call& c, int sms, double* zero_expanded, double* gathered) {
  const double flops = 2.0 * c.tokens * static_cast<double>(c.n_out) * c.k_in;
  *zero_expanded = flops / ((c.act == BSP_ACT_GELU ? 1300.0 : 1450.0) * 1e6);
  const double blocks = c.n_out / c.block;
  const double kept_per_block = c.kept_weights >= 0 ? static_cast<double>(c.kept_weights) / c.block / blocks : c.k_in;
  const double stages = blocks * (kept_per_block > 0 ? static_cast<double>((static_cast<long long>(kept_per_block) + 63) / 64) : 1.0);
  const double tiles = (c.tokens + 127) / 128;
  *gathered = tiles * (0.62 * stages + 0.45 * blocks) / sms;
}

int choose(const bsp_linear_call& c) {
  const bool z = can_zero_expanded(c), g = can_gathered(c);
  if (z && !g) return BSP_ROUTE_ZERO_EXPANDED;
  if (g && !z) return BSP_ROUTE_GATHERED;
  if (!z && !g) return 0;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  double tz, tg;
  estimate_us(c, sms, &tz, &tg);
  return tg * 1.10 < tz ? BSP_ROUTE_GATHERED : BSP_ROUTE_ZERO_EXPANDED;     // the estimate is good to about 10 %
}

int run_route(const bsp_linear_call& c, int route, cudaStream_t s) {
  void* out = c.Y ? c.Y : c.YT;
  const int ldo = c.Y ? c.ldy : c.ldyt;
  if (route == BSP_ROUTE_ZERO_EXPANDED) {
    if (!can_zero_expanded(c)) return BSP_ERR_ARG;
    const int algo = BSP_LINEAR_AUTO | (c.plan_stable ? BSP_LINEAR_PLAN_STABLE : 0) | (c.YT ? BSP_LINEAR_OUT_TRANSPOSED : 0);
    return bsp_linear_planned_ex(c.plan, c.n_out, c.k_in, c.block, c.X, c.tokens, c.ldx, c.bias, c.act, out, ldo, algo, s);
  }
  if (route == BSP_ROUTE_GATHERED) {
    if (!can_gathered(c)) return BSP_ERR_ARG;
    return bsp_linear_gathered_ex(c.gplan, c.n_out, c.k_in, c.block, c.XT, c.tokens, c.ldxt, c.bias, c.act, out, ldo,
                                  c.YT ? 1 : 0, s);
  }
  return BSP_ERR_ARG;
}

}  // namespace
}  // namespace bsp

extern "C" int bsp_linear_route(const bsp_linear_call* call, int* route) {
  using namespace bsp;
  int st = check_call(call);
  if (st != BSP_OK) return st;
  if (route == nullptr) return BSP_ERR_ARG;
  *route = choose(*call);
  return *route == 0 ? BSP_ERR_ARG : BSP_OK;       // no route: the layouts given do not fit together
}

extern "C" int bsp_linear_run(const bsp_linear_call* call, int route, int* route_taken, void* stream) {
  using namespace bsp;
  int st = check_call(call);
  if (st != BSP_OK) return st;
  if (route < BSP_ROUTE_AUTO || route > BSP_ROUTE_GATHERED) return BSP_ERR_ARG;
  if (route == BSP_ROUTE_AUTO) route = choose(*call);
  if (route == 0) return BSP_ERR_ARG;
  if (route_taken) *route_taken = route;
  return run_route(*call, route, static_cast<cudaStream_t>(stream));
}

extern "C" int bsp_linear_tune(const bsp_linear_call* call, int reps, int* best_route, float* ms_zero_expanded,
                               float* ms_gathered, void* stream) {
  using namespace bsp;
  int st = check_call(call);
  if (st != BSP_OK) return st;
  if (best_route == nullptr || reps < 1 || reps > 1000) return BSP_ERR_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  float ms[3] = {0.0f, -1.0f, -1.0f};
  cudaEvent_t a, b;
  BSP_CUDA_TRY(cudaEventCreate(&a));
  if (cudaEventCreate(&b) != cudaSuccess) { cudaEventDestroy(a); return BSP_ERR_CUDA; }
  for (int route = BSP_ROUTE_ZERO_EXPANDED; route <= BSP_ROUTE_GATHERED && st == BSP_OK; ++route) {
    if (route == BSP_ROUTE_ZERO_EXPANDED ? !can_zero_expanded(*call) : !can_gathered(*call)) continue;
    st = run_route(*call, route, s);                                 // one untimed launch first
    if (st != BSP_OK) break;
    if (cudaEventRecord(a, s) != cudaSuccess) { st = BSP_ERR_CUDA; break; }
    for (int i = 0; i < reps && st == BSP_OK; ++i) st = run_route(*call, route, s);
    if (st != BSP_OK) break;
    if (cudaEventRecord(b, s) != cudaSuccess || cudaEventSynchronize(b) != cudaSuccess ||
        cudaEventElapsedTime(&ms[route], a, b) != cudaSuccess) { st = BSP_ERR_CUDA; break; }
    ms[route] /= static_cast<float>(reps);
  }
  cudaEventDestroy(a);
  cudaEventDestroy(b);
  if (st != BSP_OK) return st;
  if (ms[1] < 0.0f && ms[2] < 0.0f) return BSP_ERR_ARG;
  *best_route = (ms[2] >= 0.0f && (ms[1] < 0.0f || ms[2] < ms[1])) ? BSP_ROUTE_GATHERED : BSP_ROUTE_ZERO_EXPANDED;
  if (ms_zero_expanded) *ms_zero_expanded = ms[1];
  if (ms_gathered) *ms_gathered = ms[2];
  return BSP_OK;
}
