// moe_plan: top-k expert ids -> per-expert counts, exclusive offsets (device prefix sum),
// the stable permutation of routed rows, the m-tile table (its length is the footprint
// x_moe of Section 6.2 of the paper) and the ordered tile list the persistent kernel's
// queues serve.
//
// The permutation is one stable counting-sort pass over the expert id.  No atomic decides
// an order: every warp ranks a fixed chunk of rows, a column scan over the per-warp
// histograms gives each warp its base rank per expert, and inside a warp rows are ranked
// by lane order, so the result is unique and reproducible.
#include "moe_dev.cuh"

namespace moe {

constexpr int kPlanThreads = 256;
constexpr int kPlanWarps = kPlanThreads / 32;

// ---------------------------------------------------------------- K1: per-warp histograms
// one warp, one chunk of kPlanChunk routed rows; h: the warp's E counters in shared memory
__device__ __forceinline__ void hist_chunk(const OpDev* __restrict__ op, Global* g, int slot, int R, int E,
                                           int chunk, int* h, int lane) {
  for (int e = lane; e < E; e += 32) h[e] = 0;
  __syncwarp();
  const int* ids = op->topk_ids;
  const int base = chunk * kPlanChunk;
  int my[kPlanChunk / 32];                    // this lane's ids of the chunk, loaded up front
#pragma unroll
  for (int it = 0; it < kPlanChunk / 32; ++it) {
    const int i = base + it * 32 + lane;
    my[it] = i < R ? ids[i] : -1;
  }
#pragma unroll
  for (int it = 0; it < kPlanChunk / 32; ++it) {
    const int i = base + it * 32 + lane;
    int id = my[it];
    if (i < R && (id < 0 || id >= E)) {
      report(&g->status, MOE_EBADID, slot, i, id, 0);
      id = -1;
    }
    const unsigned peers = __match_any_sync(0xffffffffu, id);
    if (id >= 0 && (peers & ((1u << lane) - 1)) == 0) h[id] += __popc(peers);
    __syncwarp();
  }
  int* out = op->plan_hist + (size_t)chunk * E;
  if (base < R)
    for (int e = lane; e < E; e += 32) out[e] = h[e];
}

__global__ void __launch_bounds__(kPlanThreads)
plan_hist_kernel(const OpDev* __restrict__ op, Global* g, int slot, int R, int E) {
  extern __shared__ int sm[];                 // [kPlanWarps][E]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  hist_chunk(op, g, slot, R, E, blockIdx.x * kPlanWarps + warp, sm + warp * E, lane);
}

// exclusive scan of one int per thread over a 1024-thread block
__device__ inline int block_excl_scan(int v, int* total, int* warp_sums) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    int n = __shfl_up_sync(0xffffffffu, inc, d);
    if (lane >= d) inc += n;
  }
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    int s = warp_sums[lane];
    int si = s;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      int n = __shfl_up_sync(0xffffffffu, si, d);
      if (lane >= d) si += n;
    }
    warp_sums[lane] = si - s;               // exclusive warp offsets
    if (lane == 31) warp_sums[32] = si;     // grand total
  }
  __syncthreads();
  const int res = warp_sums[warp] + inc - v;
  *total = warp_sums[32];
  __syncthreads();
  return res;
}

// ---------------------------------------------------------------- the ordered tile list of one op
// Shared-memory scratch of build_tile_list (one block of 1024 threads).
struct ListScratch {
  int warp_sums[33];
  int work[kMaxExperts], grp[kMaxExperts], moff[kMaxExperts], w0[kMaxExperts];
  int g_cnt[kMaxExperts], g_base1[kMaxExperts], g_base2[kMaxExperts];
  int ntiles;
};

// Writes the queue list of an op whose expert e holds rows [off[e], off[e] + cnt[e]) of the packed row space
// (cnt / off in shared memory), and its PlanState.
// Work tiles (the unit the queues hand out): up to `work_rows` consecutive rows of one
// expert, i.e. one or two adjacent m-tiles that share each weight tile they read.
// Dependency groups: consecutive experts holding at least kGroupWork work tiles.  The list
// is  G1(g0) G1(g1) G2(g0) G1(g2) G2(g1) ... G2(last): every down-GEMM tile comes after all
// gate/up tiles of its group and of one more group, so by the time it is claimed the tiles
// it depends on were claimed long before.
__device__ __forceinline__ int build_tile_list(int4* tile_list, PlanState* plan, const int* cnt, const int* off, int E,
                                                int NT1, int NT2, int T, int work_rows, int x_moe, int planned,
                                                int n_extra_gemm, int g1_kind = kGateUp) {
  __shared__ ListScratch ls;
  const int e = threadIdx.x;
  const int we = (e < E) ? (cnt[e] + work_rows - 1) / work_rows : 0;
  if (e < kMaxExperts) ls.work[e] = we;
  int n_work;
  const int w0 = block_excl_scan(we, &n_work, ls.warp_sums);
  if (e < E) ls.w0[e] = w0;
  __syncthreads();
  if (threadIdx.x == 0) {
    int ng = 0, acc = 0;
    for (int x = 0; x < E; ++x) {
      const int m = ls.work[x];
      ls.grp[x] = ng;
      ls.moff[x] = acc;
      acc += m;
      if (acc >= kGroupWork || x == E - 1) {
        if (acc > 0) { ls.g_cnt[ng] = acc; ++ng; }
        acc = 0;
      }
    }
    int pos = 0;
    for (int gi = 0; gi < ng; ++gi) {
      ls.g_base1[gi] = pos;
      pos += ls.g_cnt[gi] * NT1;
      if (gi >= 1) { ls.g_base2[gi - 1] = pos; pos += ls.g_cnt[gi - 1] * NT2; }
    }
    if (ng > 0) { ls.g_base2[ng - 1] = pos; pos += ls.g_cnt[ng - 1] * NT2; }
    ls.ntiles = pos;
  }
  __syncthreads();

  // Inside an expert: n-major over its work tiles, so an expert's entries of one GEMM are one
  // contiguous run of the list.  One warp per expert writes them (a popular expert has hundreds).
  for (int x = threadIdx.x >> 5; x < E; x += 32) {
    const int wx = ls.work[x];
    if (wx == 0) continue;
    const int lane = threadIdx.x & 31;
    const int gi = ls.grp[x], cx = cnt[x], ox = off[x], mx = ls.w0[x];
    const int b1 = ls.g_base1[gi] + ls.moff[x] * NT1, b2 = ls.g_base2[gi] + ls.moff[x] * NT2;
    for (int i = lane; i < wx * NT1; i += 32) {
      const int n = i / wx, j = i - n * wx;
      tile_list[b1 + i] = make_entry(g1_kind, n, mx + j, ox + j * work_rows, min(work_rows, cx - j * work_rows), x);
    }
    for (int i = lane; i < wx * NT2; i += 32) {
      const int n = i / wx, j = i - n * wx;
      tile_list[b2 + i] = make_entry(kDown, n, mx + j, ox + j * work_rows, min(work_rows, cx - j * work_rows), x);
    }
  }
  const int n_gemm = ls.ntiles;
  const int ct = combine_tile_tokens(T);
  const int n_comb = (T + ct - 1) / ct;
  for (int c = threadIdx.x; c < n_comb; c += blockDim.x)
    tile_list[n_gemm + c] = make_entry(kCombine, 0, c, c * ct, min(ct, T - c * ct), 0);
  if (threadIdx.x == 0) {
    PlanState ps;
    ps.n_mtiles = x_moe;
    ps.n_gemm_tiles = n_gemm;
    ps.n_comb_tiles = n_comb;
    ps.planned = planned;                   // a plan with a rejected id leaves the slot without tiles to run
    ps.n_extra_gemm = n_extra_gemm;
    ps.pad[0] = ps.pad[1] = ps.pad[2] = 0;
    *plan = ps;
  }
  __syncthreads();
  return n_gemm;
}

// ---------------------------------------------------------------- K2: scans + tile table + tile list
// the whole block of 1024 threads
__device__ __forceinline__ void scan_body(const OpDev* __restrict__ op, int n_chunks, int R, int E, int NT1, int NT2,
                                          int T, int work_rows) {
  __shared__ int warp_sums[33];
  __shared__ int s_cnt[kMaxExperts], s_off[kMaxExperts];
  __shared__ int s_part[1024];
  const int e = threadIdx.x;

  // column sums of the per-warp histograms, the device prefix sum over experts, then the base
  // rank of every (warp chunk, expert).  Reads and writes use different arrays so that the
  // loads of a column do not wait on the stores.
  const int* hist = op->plan_hist;        // no __restrict__: the one-block plan wrote it earlier in the same kernel
  int* base = op->plan_base;
  // the 1024 threads split every expert's column into `parts` chunk ranges
  const int parts = max(1, 1024 / E);
  const int part = threadIdx.x / E, pe = threadIdx.x % E;
  const int cpp = (n_chunks + parts - 1) / parts;
  const int c0 = min(n_chunks, part * cpp), c1 = min(n_chunks, c0 + cpp);
  int psum = 0;
  if (part < parts) {
#pragma unroll 32
    for (int c = c0; c < c1; ++c) psum += hist[(size_t)c * E + pe];
    s_part[part * E + pe] = psum;
  }
  __syncthreads();
  int cnt = 0;
  if (e < E)
    for (int p = 0; p < parts; ++p) cnt += s_part[p * E + e];
  int total;
  const int off = block_excl_scan(cnt, &total, warp_sums);       // device prefix sum over experts
  if (e < E) {
    op->counts[e] = cnt;
    op->offsets[e] = off;
    s_cnt[e] = cnt;
    s_off[e] = off;
  }
  if (e == 0) op->offsets[E] = total;
  // rows with a rejected expert id take no packed position: the tail of the permutation that no row
  // will claim is marked, so that nothing downstream mistakes stale memory for an index
  for (int p = total + (int)threadIdx.x; p < R; p += (int)blockDim.x) op->sorted_to_flat[p] = -1;
  __syncthreads();
  if (part < parts) {
    int run = s_off[pe];
    for (int p = 0; p < part; ++p) run += s_part[p * E + pe];
#pragma unroll 32
    for (int c = c0; c < c1; ++c) {
      const int v = hist[(size_t)c * E + pe];
      base[(size_t)c * E + pe] = run;
      run += v;
    }
  }

  // m-tiles: ceil(m_e / M_t) per expert with rows (the footprint x_moe)
  const int me = (e < E) ? (cnt + kTileM - 1) / kTileM : 0;
  int x_moe;
  const int m0 = block_excl_scan(me, &x_moe, warp_sums);
  if (e < E) {
    for (int j = 0; j < me; ++j) {
      MTile t;
      t.expert = e;
      t.row0 = off + j * kTileM;
      t.rows = min(kTileM, cnt - j * kTileM);
      t.pad = 0;
      op->mtiles[m0 + j] = t;
    }
  }
  __syncthreads();

  build_tile_list(op->tile_list, op->plan, s_cnt, s_off, E, NT1, NT2, T, work_rows, x_moe, total == R ? 1 : 0, 0);
}

__global__ void __launch_bounds__(1024)
plan_scan_kernel(const OpDev* __restrict__ op, int n_chunks, int R, int E, int NT1, int NT2,
                 int T, int work_rows) {
  scan_body(op, n_chunks, R, E, NT1, NT2, T, work_rows);
}

// ---------------------------------------------------------------- K3: stable scatter
// one warp, one chunk; run: the warp's E running ranks in shared memory
__device__ __forceinline__ void scatter_chunk(const OpDev* __restrict__ op, int R, int E, int chunk, int* run, int lane) {
  const int base = chunk * kPlanChunk;
  if (base >= R) return;
  const int* src = op->plan_base + (size_t)chunk * E;
  for (int e = lane; e < E; e += 32) run[e] = src[e];
  __syncwarp();
  const int* ids = op->topk_ids;
  int* s2f = op->sorted_to_flat;
  int* f2s = op->flat_to_sorted;
  int my[kPlanChunk / 32];
#pragma unroll
  for (int it = 0; it < kPlanChunk / 32; ++it) {
    const int i = base + it * 32 + lane;
    my[it] = i < R ? ids[i] : -1;
  }
#pragma unroll
  for (int it = 0; it < kPlanChunk / 32; ++it) {
    const int i = base + it * 32 + lane;
    int id = my[it];
    if (id < 0 || id >= E) id = -1;         // reported by the histogram pass
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
    } else if (i < R) {
      f2s[i] = -1;                          // a rejected id: the row has no packed position
    }
  }
}

__global__ void __launch_bounds__(kPlanThreads)
plan_scatter_kernel(const OpDev* __restrict__ op, int R, int E) {
  extern __shared__ int sm[];                 // [kPlanWarps][E] running rank per expert
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  scatter_chunk(op, R, E, blockIdx.x * kPlanWarps + warp, sm + warp * E, lane);
}

// ---------------------------------------------------------------- small ops: the three passes in one block
// An op of at most kSmallChunks chunks (a decode batch) is planned by ONE block of 32 warps: the
// histogram scratch written by the first pass is read back by the same block, so two launches and
// their gaps go away (they are about half of a small plan's time).
constexpr int kSmallChunks = 32;
constexpr int kSmallMaxExperts = 256;

__global__ void __launch_bounds__(1024)
plan_small_kernel(const OpDev* __restrict__ op, Global* g, int slot, int n_chunks, int R, int E, int NT1, int NT2,
                  int T, int work_rows) {
  extern __shared__ int sm[];                 // [32 warps][E]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp < n_chunks) hist_chunk(op, g, slot, R, E, warp, sm + warp * E, lane);
  __threadfence_block();
  __syncthreads();
  scan_body(op, n_chunks, R, E, NT1, NT2, T, work_rows);
  __threadfence_block();
  __syncthreads();
  if (warp < n_chunks) scatter_chunk(op, R, E, warp, sm + warp * E, lane);
}

// ---------------------------------------------------------------- masked layout
// The activations already sit in per-expert slabs of slab_rows rows; counts[e] (an input here) says how many
// rows of slab e are valid.  Nothing is permuted: the plan is the exclusive prefix sum for `offsets`, the
// m-tile table (first row of a tile = e * slab_rows + 128 j) and the queue list over the slabs' valid rows.
__global__ void __launch_bounds__(1024)
plan_masked_kernel(const OpDev* __restrict__ op, Global* g, int slot, int E, int NT1, int NT2, int slab_rows, int work_rows) {
  __shared__ int warp_sums[33];
  __shared__ int s_cnt[kMaxExperts], s_off[kMaxExperts];
  const int e = threadIdx.x;
  int cnt = 0;
  if (e < E) {
    cnt = op->counts[e];
    if (cnt < 0 || cnt > slab_rows) {        // a count the slab cannot hold: reported, the slab is left out
      report(&g->status, MOE_EBOUNDS, slot, e, cnt, 4);
      cnt = 0;
    }
    s_cnt[e] = cnt;
    s_off[e] = e * slab_rows;
  }
  int total;
  const int off = block_excl_scan(cnt, &total, warp_sums);
  if (e < E) op->offsets[e] = off;
  if (e == 0) op->offsets[E] = total;
  const int me = (e < E) ? (cnt + kTileM - 1) / kTileM : 0;
  int x_moe;
  const int m0 = block_excl_scan(me, &x_moe, warp_sums);
  if (e < E) {
    for (int j = 0; j < me; ++j) {
      MTile t;
      t.expert = e;
      t.row0 = e * slab_rows + j * kTileM;
      t.rows = min(kTileM, cnt - j * kTileM);
      t.pad = 0;
      op->mtiles[m0 + j] = t;
    }
  }
  __syncthreads();
  build_tile_list(op->tile_list, op->plan, s_cnt, s_off, E, NT1, NT2, 0, work_rows, x_moe, 1, 0, kGateUpDirect);
}

cudaError_t launch_plan_masked(const OpDev* d_op, Global* g, int slot, int E, int NT1, int NT2, int slab_rows, int work_rows,
                               cudaStream_t stream) {
  plan_masked_kernel<<<1, 1024, 0, stream>>>(d_op, g, slot, E, NT1, NT2, slab_rows, work_rows);
  return cudaGetLastError();
}

// ---------------------------------------------------------------- the paired form of a decode + prefill op
// Two ops of one launch that share their expert weights can share weight tiles too.  The paired form puts
// the routed rows of both into ONE packed row space -- per expert the prefill rows (in their plan's order)
// followed by the decode rows (in theirs) -- and cuts it into two queue lists: per expert, the decode list
// takes the decode rows plus the ragged tail of the prefill rows just before them if it fits into the decode
// rows' last tile of `carrier_rows` rows ("carrier" tiles: claimed with decode priority, they stream a weight
// tile once for rows of both ops); the prefill list takes the rest.  Nothing about a row's arithmetic depends on the
// tile it sits in, so the outputs are those of the unpaired ops, bit for bit.
//   dp / pp: the paired descriptors (their PlanStates and lists are written here), d / p: the plain ones,
//   whose counts and offsets the two moe_plan calls have written earlier on the stream.
__global__ void __launch_bounds__(1024)
plan_pair_kernel(const OpDev* dp, const OpDev* pp, const OpDev* d, const OpDev* p, int E, int NT1, int NT2,
                 int work_rows, int carrier_rows) {
  __shared__ int cnt_d[kMaxExperts], off_d[kMaxExperts], cnt_p[kMaxExperts], off_p[kMaxExperts];
  const int e = threadIdx.x;
  if (e < E) {
    const int cd = d->counts[e], cp = p->counts[e];
    const int moff = d->offsets[e] + p->offsets[e];
    // the carrier takes the ragged tail of the prefill rows (what is left over after the prefill op's full work
    // tiles) when that tail fits beside the decode rows: a prefill tile less to run.  A tail that does not fit
    // stays where it is -- moving part of it would make the carrier heavier and save nothing.
    const int room = cd > 0 ? (cd + carrier_rows - 1) / carrier_rows * carrier_rows - cd : 0;
    const int tail = cp % max(work_rows, carrier_rows);
    const int take = tail <= room ? tail : 0;
    cnt_p[e] = cp - take;
    off_p[e] = moff;
    cnt_d[e] = cd + take;
    off_d[e] = moff + cp - take;
  }
  __syncthreads();
  const int ok = (d->plan->planned && p->plan->planned) ? 1 : 0;
  // a carrier taller than the kernel's work tile (e4m3: 128 rows) is cut into work tiles that follow one another
  const int n_dec = build_tile_list(dp->tile_list, dp->plan, cnt_d, off_d, E, NT1, NT2, d->n_tokens,
                                    min(carrier_rows, work_rows), d->plan->n_mtiles, ok, 0);
  // every GEMM entry of the decode list may carry prefill rows: the prefill op is complete when they are too
  build_tile_list(pp->tile_list, pp->plan, cnt_p, off_p, E, NT1, NT2, p->n_tokens, work_rows, p->plan->n_mtiles, ok,
                  n_dec);
}

// the shared row space's permutation: for each op, flat routed index -> packed row, and packed row -> flat
// index tagged with the slot the row belongs to
__global__ void __launch_bounds__(256)
plan_pair_scatter_kernel(const OpDev* d, const OpDev* p, int* gather_m, int* comb_d, int* comb_p, int Rd, int Rp, int E,
                         int slot_d, int slot_p) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < Rd) {
    const int e = d->topk_ids[i], ps = d->flat_to_sorted[i];
    int m = -1;
    if (e >= 0 && e < E && ps >= 0) {
      m = ps + p->offsets[e + 1];               // behind the expert's prefill rows
      gather_m[m] = i | (slot_d << kRowSlotShift);
    }
    comb_d[i] = m;
  } else if (i < Rd + Rp) {
    const int j = i - Rd;
    const int e = p->topk_ids[j], ps = p->flat_to_sorted[j];
    int m = -1;
    if (e >= 0 && e < E && ps >= 0) {
      m = ps + d->offsets[e];                   // shifted by the decode rows of the experts before
      gather_m[m] = j | (slot_p << kRowSlotShift);
    }
    comb_p[j] = m;
  }
}

cudaError_t launch_plan_pair(const OpDev* dp, const OpDev* pp, const OpDev* d, const OpDev* p, int* gather_m, int* comb_d,
                             int* comb_p, int Rd, int Rp, int E, int NT1, int NT2, int work_rows, int carrier_rows,
                             int slot_d, int slot_p, cudaStream_t stream) {
  plan_pair_kernel<<<1, 1024, 0, stream>>>(dp, pp, d, p, E, NT1, NT2, work_rows, carrier_rows);
  const int n = Rd + Rp;
  if (n > 0)
    plan_pair_scatter_kernel<<<(n + 255) / 256, 256, 0, stream>>>(d, p, gather_m, comb_d, comb_p, Rd, Rp, E, slot_d, slot_p);
  return cudaGetLastError();
}

cudaError_t prepare_plan_kernels() {
  return cudaFuncSetAttribute(plan_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              kSmallChunks * kSmallMaxExperts * (int)sizeof(int));
}

cudaError_t launch_plan(const OpDev* d_op, Global* g, int slot, int T, int k, int E, int NT1,
                        int NT2, int work_rows, cudaStream_t stream) {
  const int R = T * k;
  const int n_chunks = (R + kPlanChunk - 1) / kPlanChunk;
  const int blocks = (n_chunks + kPlanWarps - 1) / kPlanWarps;
  const size_t smem = (size_t)kPlanWarps * E * sizeof(int);
  if (n_chunks <= kSmallChunks && E <= kSmallMaxExperts) {
    plan_small_kernel<<<1, 1024, (size_t)kSmallChunks * E * sizeof(int), stream>>>(d_op, g, slot, n_chunks, R, E, NT1, NT2, T,
                                                                                 work_rows);
    return cudaGetLastError();
  }
  if (blocks > 0) plan_hist_kernel<<<blocks, kPlanThreads, smem, stream>>>(d_op, g, slot, R, E);
  plan_scan_kernel<<<1, 1024, 0, stream>>>(d_op, n_chunks, R, E, NT1, NT2, T, work_rows);
  if (blocks > 0) plan_scatter_kernel<<<blocks, kPlanThreads, smem, stream>>>(d_op, R, E);
  return cudaGetLastError();
}

}  // namespace moe
