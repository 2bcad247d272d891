// moe_route: the router ahead of the plan step -- per token the k experts with the largest logits
// and the router weights softmax(logits) renormalised over those k (the router step of the MoE
// module of Section 2.1 of the paper; the paper does not fix the arithmetic, this is the
// softmax -> top-k -> renormalise form of the seeded workloads).
//
// One warp per token.  Each lane holds the logits e = lane, lane + 32, ... in registers (E <= 1024);
// k rounds of a warp arg-max pick the experts in order of decreasing logit, ties to the lower
// expert id, which is the order of decreasing softmax probability.  The weights need no sum over
// all E experts: exp(z_j - z_max) / sum over the chosen k of the same, the common denominator
// cancels.  No workspace, no context.
#include "moe_dev.cuh"

namespace moe {

constexpr int kRouteMaxE = 1024;
constexpr int kRouteWarps = 8;

__global__ void __launch_bounds__(kRouteWarps * 32) route_kernel(const float* __restrict__ logits, int T, int E, int k,
                                                                 int* __restrict__ ids, float* __restrict__ w) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x * kRouteWarps + warp;
  if (t >= T) return;
  const float* z = logits + (size_t)t * E;
  constexpr int kPer = kRouteMaxE / 32;
  float v[kPer];
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int e = lane + 32 * i;
    v[i] = e < E ? z[e] : -INFINITY;
  }
  unsigned used = 0;                       // bit i: this lane's element i is taken
  float zmax = 0.f, mine = 0.f, sum = 0.f; // lane j keeps exp(z - zmax) of the j-th pick (k <= 32)
  for (int j = 0; j < k; ++j) {
    float best = -INFINITY;
    int arg = 0x7fffffff;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
      const int e = lane + 32 * i;
      if (e < E && !((used >> i) & 1u) && (v[i] > best || arg == 0x7fffffff)) { best = v[i]; arg = e; }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {     // arg-max over the warp, ties to the lower expert id
      const float ob = __shfl_xor_sync(0xffffffffu, best, d);
      const int oa = __shfl_xor_sync(0xffffffffu, arg, d);
      if (oa != 0x7fffffff && (arg == 0x7fffffff || ob > best || (ob == best && oa < arg))) { best = ob; arg = oa; }
    }
    if ((arg & 31) == lane) used |= 1u << (arg >> 5);
    if (j == 0) zmax = best;
    const float p = expf(best - zmax);
    sum += p;
    if (lane == j) mine = p;
    if (lane == 0) ids[(size_t)t * k + j] = arg;
  }
  if (lane < k) w[(size_t)t * k + lane] = mine / sum;
}

}  // namespace moe

extern "C" int moe_route(const float* logits, int32_t n_tokens, int32_t n_experts, int32_t top_k,
                         int32_t* topk_ids, float* topk_w, void* stream) {
  using namespace moe;
  if (n_tokens < 0 || n_experts < 1 || n_experts > kRouteMaxE || top_k < 1 || top_k > 32 || top_k > n_experts)
    return MOE_EINVAL;
  if (n_tokens == 0) return MOE_OK;
  if (!logits || !topk_ids || !topk_w) return MOE_EINVAL;
  const int blocks = (n_tokens + kRouteWarps - 1) / kRouteWarps;
  route_kernel<<<blocks, kRouteWarps * 32, 0, static_cast<cudaStream_t>(stream)>>>(logits, n_tokens, n_experts, top_k,
                                                                                  topk_ids, topk_w);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ECUDA;
}
