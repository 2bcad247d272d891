// moe_plan_static: the plan step (counts, exclusive offsets, stable permutation) for callers
// that must not allocate.  It needs no context and no workspace: the per-warp histogram
// scratch that moe_plan keeps in the caller's workspace lives here in a fixed device array
// that is part of the library image, so every GPU that loads the library carries it (128 KB)
// until the process exits.
//
// Who needs this: code that runs where a device allocation is off limits -- a serving loop
// whose memory was handed in full to another allocator, a callback that may not make calls
// that can synchronise the device (cudaMalloc / cudaFree can), a sandboxed plug-in that only
// gets the buffers it is passed.  Such a caller still owns inputs and outputs; only the
// scratch is ours.
//
// The array's name is a host-side handle in host code, not a device address, so the address
// is looked up with cudaGetSymbolAddress and that pointer is what the kernels receive.  The
// first look-up on a device may load the library's device code; make that first call outside
// any stream capture.
//
// All calls share the one array and it keeps the last call's contents.  Nothing in it has
// to start at zero (every entry a call reads was written by the same call), but two calls
// whose kernels overlap on the GPU (different streams, or different host threads) would
// race on it: serialise them.
#include "moe_dev.cuh"

namespace moe {

constexpr int kStaticMaxRows = MOE_PLAN_STATIC_MAX_ROWS;
constexpr int kStaticMaxExperts = MOE_PLAN_STATIC_MAX_EXPERTS;
constexpr int kStaticChunkRows = 256;                    // routed rows ranked by one warp
constexpr int kStaticChunks = kStaticMaxRows / kStaticChunkRows;
constexpr int kStaticThreads = 256;
constexpr int kStaticWarps = kStaticThreads / 32;

static __device__ __align__(256) int g_plan_scratch[kStaticChunks * kStaticMaxExperts];

// per-warp histogram of a fixed chunk of routed rows -> hist[chunk][E]
__global__ void __launch_bounds__(kStaticThreads)
static_hist_kernel(const int* __restrict__ ids, int* __restrict__ hist, int R, int E) {
  __shared__ int sm[kStaticWarps * kStaticMaxExperts];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunk = blockIdx.x * kStaticWarps + warp;
  const int base = chunk * kStaticChunkRows;
  int* h = sm + warp * E;
  for (int e = lane; e < E; e += 32) h[e] = 0;
  __syncwarp();
  for (int it = 0; it < kStaticChunkRows / 32; ++it) {
    const int i = base + it * 32 + lane;
    int id = -1;
    if (i < R) {
      id = ids[i];
      if (id < 0 || id >= E) id = -1;
    }
    const unsigned peers = __match_any_sync(0xffffffffu, id);
    if (id >= 0 && (peers & ((1u << lane) - 1)) == 0) h[id] += __popc(peers);
    __syncwarp();
  }
  if (base < R)
    for (int e = lane; e < E; e += 32) hist[(size_t)chunk * E + e] = h[e];
}

// one block: column scan over chunks (base rank of every chunk per expert), then the
// exclusive prefix sum over experts
__global__ void __launch_bounds__(kStaticMaxExperts)
static_scan_kernel(int* __restrict__ hist, int n_chunks, int E, int* __restrict__ counts,
                   int* __restrict__ offsets) {
  __shared__ int s[kStaticMaxExperts];
  const int e = threadIdx.x;
  int cnt = 0;
  if (e < E) {
    for (int c = 0; c < n_chunks; ++c) {
      const int v = hist[(size_t)c * E + e];
      hist[(size_t)c * E + e] = cnt;
      cnt += v;
    }
  }
  s[e] = cnt;
  __syncthreads();
  for (int d = 1; d < kStaticMaxExperts; d <<= 1) {       // inclusive scan in shared memory
    const int v = e >= d ? s[e - d] : 0;
    __syncthreads();
    s[e] += v;
    __syncthreads();
  }
  const int off = s[e] - cnt;
  if (e < E) {
    counts[e] = cnt;
    offsets[e] = off;
    for (int c = 0; c < n_chunks; ++c) hist[(size_t)c * E + e] += off;
  }
  if (e == E - 1) offsets[E] = s[e];
}

// stable scatter: rows of a warp's chunk are ranked in lane order
__global__ void __launch_bounds__(kStaticThreads)
static_scatter_kernel(const int* __restrict__ ids, const int* __restrict__ hist, int R, int E,
                      int* __restrict__ s2f, int* __restrict__ f2s) {
  __shared__ int sm[kStaticWarps * kStaticMaxExperts];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunk = blockIdx.x * kStaticWarps + warp;
  const int base = chunk * kStaticChunkRows;
  if (base >= R) return;
  int* run = sm + warp * E;
  for (int e = lane; e < E; e += 32) run[e] = hist[(size_t)chunk * E + e];
  __syncwarp();
  for (int it = 0; it < kStaticChunkRows / 32; ++it) {
    const int i = base + it * 32 + lane;
    int id = -1;
    if (i < R) {
      id = ids[i];
      if (id < 0 || id >= E) id = -1;
    }
    const unsigned peers = __match_any_sync(0xffffffffu, id);
    const unsigned before = peers & ((1u << lane) - 1);
    int p = -1;
    if (id >= 0) p = run[id] + __popc(before);
    __syncwarp();
    if (id >= 0 && before == 0) run[id] += __popc(peers);
    __syncwarp();
    if (p >= 0 && p < R) {
      s2f[p] = i;
      f2s[i] = p;
    }
  }
}

// Device address of the scratch array on the current device.  Looked up on every call: a cached
// pointer would dangle once the caller resets the device (the array then moves with the reloaded
// module), and after the first call the look-up is a table read.
static int scratch_on_current_device(int** out) {
  void* p = nullptr;
  const cudaError_t e = cudaGetSymbolAddress(&p, g_plan_scratch);
  if (e != cudaSuccess || p == nullptr) return MOE_ECUDA;
  *out = static_cast<int*>(p);
  return MOE_OK;
}

}  // namespace moe

extern "C" int moe_plan_static(const int32_t* topk_ids, int32_t n_tokens, int32_t top_k,
                               int32_t n_experts, int32_t* counts, int32_t* offsets,
                               int32_t* sorted_to_flat, int32_t* flat_to_sorted, void* stream) {
  using namespace moe;
  if (n_tokens < 0 || top_k < 1 || n_experts < 1 || !counts || !offsets) return MOE_EINVAL;
  if (n_experts > kStaticMaxExperts) return MOE_ENOSPC;        // beyond the fixed scratch
  const long long R64 = (long long)n_tokens * top_k;
  if (R64 > kStaticMaxRows) return MOE_ENOSPC;
  const int R = (int)R64;
  if (R > 0 && (!topk_ids || !sorted_to_flat || !flat_to_sorted)) return MOE_EINVAL;
  int* scratch = nullptr;
  const int rc = scratch_on_current_device(&scratch);
  if (rc != MOE_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int n_chunks = (R + kStaticChunkRows - 1) / kStaticChunkRows;
  const int blocks = (n_chunks + kStaticWarps - 1) / kStaticWarps;
  if (blocks > 0) static_hist_kernel<<<blocks, kStaticThreads, 0, st>>>(topk_ids, scratch, R, n_experts);
  static_scan_kernel<<<1, kStaticMaxExperts, 0, st>>>(scratch, n_chunks, n_experts, counts, offsets);
  if (blocks > 0)
    static_scatter_kernel<<<blocks, kStaticThreads, 0, st>>>(topk_ids, scratch, R, n_experts,
                                                             sorted_to_flat, flat_to_sorted);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ECUDA;
}
