// moe_combine: the stand-alone post-processing kernel (HBM-bound gather-reduce).
#include "moe_combine.cuh"

namespace moe {

constexpr int kCombThreads = 256;
constexpr int kCombTokensPerBlock = 4;

__global__ void __launch_bounds__(kCombThreads)
combine_kernel(const OpDev* __restrict__ op, int T, int k, int H) {
  if (op->plan->planned == 0) return;          // the slot's plan was rejected: there is no permutation to follow
  const int t0 = blockIdx.x * kCombTokensPerBlock;
  const int t1 = min(T, t0 + kCombTokensPerBlock);
  if (t0 < t1) combine_tokens(op, t0, t1, k, H, threadIdx.x, kCombThreads);
}

cudaError_t launch_combine(const OpDev* d_op, int T, int k, int H, cudaStream_t stream) {
  if (T <= 0) return cudaSuccess;
  const int blocks = (T + kCombTokensPerBlock - 1) / kCombTokensPerBlock;
  combine_kernel<<<blocks, kCombThreads, 0, stream>>>(d_op, T, k, H);
  return cudaGetLastError();
}

}  // namespace moe
