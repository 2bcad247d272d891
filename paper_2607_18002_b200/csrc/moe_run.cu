// moe_run: the persistent expert kernel (the adaptive persistent kernel of Section 4 of the
// paper, rebuilt for sm_100a).
//
// One CTA per SM, 6 warps with fixed roles:
//   warp 0     scheduler + producer.  At every tile boundary it reads the decode budget
//              word and the two queue heads, claims the next tile (decode first for CTAs
//              below the budget, prefill first for the others, each falling back to the
//              other class: Sections 4.2 and 5.4), hands the tile to the other warps
//              through a shared-memory ring guarded by mbarriers (the hand-off of
//              Section 4.3: the first pipeline warp decides, later warps follow), waits for
//              the tile's dependencies, then feeds the pipeline: weight tiles by tiled TMA,
//              activation rows by TMA gather4 through the permutation.
//   warp 1     issues tcgen05.mma (128 x 256 x 16, bf16 -> fp32) into one of two TMEM
//              accumulators; tcgen05.commit releases pipeline stages and publishes the
//              accumulator.
//   warps 2-5  epilogue: tcgen05.ld, SwiGLU (gate/up tiles), bf16 stores, then the release
//              of dependency counters, the op's done word and the tile log.  They also run
//              the combine tiles.
// A phase switch happens only between tiles, so no accumulator, TMA transaction or buffer is
// live across it (Section 4.2) and results are independent of the schedule.
//
// Every wait (mbarrier, dependency counter, ready word) is bounded: when it runs out the
// kernel records MOE_ETIMEOUT, raises the abort word, and all CTAs drain and return.
#include "moe_combine.cuh"
#include "moe_ptx.cuh"

namespace moe {

constexpr int kThreads = 192;
constexpr int kABytes = kTileM * kBlockK * 2;          // 16 KB activations per stage
constexpr int kBHalfBytes = 128 * kBlockK * 2;         // 16 KB per 128 weight rows
constexpr int kBBytes = 2 * kBHalfBytes;               // 32 KB weights per stage
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kRing = 4;                               // tile-info ring depth
constexpr int kAccCols = 256;                          // TMEM columns per accumulator
constexpr int kEnd = -1;

struct TileInfo {
  int kind, slot, tile, m, row0, rows, n, kblocks, expert, cls;
  unsigned long long t_claim;
};

struct SharedCtl {
  unsigned long long full[kStages], empty[kStages];
  unsigned long long tfull[2], tempty[2];
  unsigned long long ifull[kRing], iempty[kRing];
  TileInfo info[kRing];
  unsigned tmem_base;
  int epi_fail;
  int n_cls[2];
  int cls_slot[2][kMaxOps];
  unsigned cum[2][kMaxOps + 1];
};

constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + sizeof(SharedCtl);

// ------------------------------------------------------------------ bounded waits
struct Ctx {
  const RunArgs* a;
  Status* st;
};

__device__ __forceinline__ bool aborted(const Ctx& c) { return ld_volatile(&c.st->abort) != 0; }

// where: a small code telling which wait gave up (reported in detail[0])
__device__ __noinline__ bool mbar_wait_slow(const Ctx& c, void* bar, unsigned parity, int where) {
  unsigned long long t0 = 0;
  for (unsigned it = 1;; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 63u) == 0) {
      if (aborted(c)) return false;
      const unsigned long long now = gtime_ns();
      if (t0 == 0) t0 = now;
      else if ((long long)(now - t0) > c.a->wait_ns) {
        report(c.st, MOE_ETIMEOUT, where, (int)blockIdx.x, (int)threadIdx.x, (int)parity);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait(const Ctx& c, void* bar, unsigned parity, int where) {
  if (mbar_try(bar, parity)) return true;
  return mbar_wait_slow(c, bar, parity, where);
}

// spin until *p >= target (acquire); one thread
__device__ __noinline__ bool wait_counter(const Ctx& c, const int* p, int target, int where) {
  unsigned long long t0 = 0;
  for (unsigned it = 0;; ++it) {
    if (ld_acquire(p) >= target) return true;
    if (it > 16) __nanosleep(64);
    if ((it & 63u) == 63u) {
      if (aborted(c)) return false;
      const unsigned long long now = gtime_ns();
      if (t0 == 0) t0 = now;
      else if ((long long)(now - t0) > c.a->wait_ns) {
        report(c.st, MOE_ETIMEOUT, where, (int)blockIdx.x, target, ld_acquire(p));
        return false;
      }
    }
  }
}

// ------------------------------------------------------------------ queues
__device__ __forceinline__ int op_total_tiles(const OpDev* op, int fuse) {
  return op->plan->n_gemm_tiles + (fuse ? op->plan->n_comb_tiles : 0);
}

__device__ inline bool op_ready(const RunArgs* a, const OpDev* op) {
  if (op->ready != nullptr && ld_acquire_sys(op->ready) == 0) return false;
  if (op->after_op >= 0 && ld_acquire(&a->ops[op->after_op].run->done) == 0) return false;
  return true;
}

// 1: claimed (ti filled), 0: queue exhausted, -1: head op not ready
__device__ inline int try_claim(const RunArgs* a, SharedCtl* sc, RunHead* rh, int cls, TileInfo& ti) {
  const int n = sc->n_cls[cls];
  if (n == 0) return 0;
  const unsigned total = sc->cum[cls][n];
  unsigned h = *reinterpret_cast<volatile unsigned*>(&rh->heads[cls]);
  while (true) {
    if (h >= total) return 0;
    int i = 0;
    while (h >= sc->cum[cls][i + 1]) ++i;
    const int slot = sc->cls_slot[cls][i];
    const OpDev* op = &a->ops[slot];
    if (!op_ready(a, op)) return -1;
    const unsigned old = atomicCAS(&rh->heads[cls], h, h + 1);
    if (old == h) {
      const int local = (int)(h - sc->cum[cls][i]);
      const int entry = op->tile_list[local];
      ti.kind = tile_kind(entry);
      ti.slot = slot;
      ti.tile = local;
      ti.m = tile_m(entry);
      ti.n = tile_n(entry);
      ti.cls = cls;
      if (ti.kind == kCombine) {
        ti.row0 = ti.m * kCombineTokens;
        ti.rows = min(kCombineTokens, op->n_tokens - ti.row0);
        ti.expert = 0;
        ti.kblocks = 0;
      } else {
        const MTile mt = op->mtiles[ti.m];
        ti.row0 = mt.row0;
        ti.rows = mt.rows;
        ti.expert = mt.expert;
        ti.kblocks = (ti.kind == kGateUp ? a->H : a->I) / kBlockK;
      }
      return 1;
    }
    h = old;
  }
}

// The decision at a tile boundary.  Returns with ti.kind == kEnd when nothing is left (or
// the run was aborted).
__device__ inline void claim_next(const Ctx& c, SharedCtl* sc, RunHead* rh, TileInfo& ti) {
  const RunArgs* a = c.a;
  unsigned long long t0 = 0;
  for (unsigned it = 0;; ++it) {
    if (aborted(c)) break;
    const int q = ld_volatile(&a->g->budget);
    const int first = ((int)blockIdx.x < q) ? MOE_CLASS_DECODE : MOE_CLASS_PREFILL;
    const int r1 = try_claim(a, sc, rh, first, ti);
    if (r1 == 1) { ti.t_claim = gtime_ns(); return; }
    const int r2 = try_claim(a, sc, rh, 1 - first, ti);
    if (r2 == 1) { ti.t_claim = gtime_ns(); return; }
    if (r1 == 0 && r2 == 0) break;
    __nanosleep(256);                         // an op exists but is not ready yet
    if ((it & 15u) == 15u) {
      const unsigned long long now = gtime_ns();
      if (t0 == 0) t0 = now;
      else if ((long long)(now - t0) > a->wait_ns) {
        report(c.st, MOE_ETIMEOUT, 1, (int)blockIdx.x, r1, r2);
        break;
      }
    }
  }
  ti.kind = kEnd;
}

// Publishing a finished tile: dependency counter, op completion, done word, log.
// Called by one thread after all writers of the tile have fenced and synchronised.
__device__ inline void commit_tile(const Ctx& c, RunHead* rh, const TileInfo& ti) {
  const RunArgs* a = c.a;
  OpDev* op = &a->ops[ti.slot];
  __threadfence();
  fence_async_proxy();
  const unsigned long long t_commit = a->log_cap > 0 ? gtime_ns() : 0ull;   // before it is published
  if (ti.kind == kGateUp) atomicAdd(&op->g1_done[ti.m], 1);
  if (ti.kind != kCombine) atomicAdd(&op->run->gemm_done, 1);
  const int done = atomicAdd(&op->run->tiles_done, 1) + 1;
  if (done == op_total_tiles(op, a->fuse_combine)) {
    __threadfence();
    atomicExch(&op->run->done, 1);
    if (op->done != nullptr) st_release_sys(op->done, 1u);
  }
  if (a->log_cap > 0) {
    const unsigned idx = atomicAdd(&rh->log_count, 1u);
    if (idx < (unsigned)a->log_cap) {
      moe_tile_rec_t r;
      r.t_claim = ti.t_claim;
      r.t_commit = t_commit;
      r.slot = ti.slot;
      r.tile = ti.tile;
      r.cls = (int16_t)ti.cls;
      r.kind = (int16_t)ti.kind;
      r.cta = (int16_t)blockIdx.x;
      unsigned smid;
      asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
      r.sm = (int16_t)smid;
      a->log[idx] = r;
    }
  }
}

__device__ inline void build_queues(const RunArgs* a, SharedCtl* sc) {
  sc->n_cls[0] = sc->n_cls[1] = 0;
  sc->cum[0][0] = sc->cum[1][0] = 0;
  for (int i = 0; i < a->n_ops; ++i) {
    const int slot = a->slots[i];
    const OpDev* op = &a->ops[slot];
    const int cls = op->cls;
    const int j = sc->n_cls[cls]++;
    sc->cls_slot[cls][j] = slot;
    sc->cum[cls][j + 1] = sc->cum[cls][j] + (unsigned)op_total_tiles(op, a->fuse_combine);
  }
}

__device__ __forceinline__ float silu_mul(float g, float u) {
  return g / (1.0f + __expf(-g)) * u;
}

// ------------------------------------------------------------------ the persistent kernel
__global__ void __launch_bounds__(kThreads, 1) moe_apk_kernel(const __grid_constant__ RunArgs args,
                                                              RunHead* rh) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* stages = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  SharedCtl* sc = reinterpret_cast<SharedCtl*>(stages + (size_t)kStages * kStageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  Ctx c{&args, &args.g->status};

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&sc->full[s], 1); mbar_init(&sc->empty[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&sc->tfull[s], 1); mbar_init(&sc->tempty[s], 128); }
    for (int s = 0; s < kRing; ++s) { mbar_init(&sc->ifull[s], 1); mbar_init(&sc->iempty[s], 2); }
    build_queues(&args, sc);
    sc->epi_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_proxy();
  }
  if (warp == 1) {   // TMEM: both accumulators (512 columns); this warp also frees them
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&sc->tmem_base)),
                 "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const unsigned tmem = sc->tmem_base;

  if (warp == 0) {
    // ============================================================ scheduler + producer
    int stage = 0, islot = 0;
    unsigned ph = 0, iph = 0;
    while (true) {
      if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->iempty[islot], iph ^ 1u, 2))) break;
      TileInfo ti;
      ti.kind = kEnd;
      if (lane == 0) claim_next(c, sc, rh, ti);
      ti.kind = __shfl_sync(0xffffffffu, ti.kind, 0);
      ti.slot = __shfl_sync(0xffffffffu, ti.slot, 0);
      ti.m = __shfl_sync(0xffffffffu, ti.m, 0);
      ti.n = __shfl_sync(0xffffffffu, ti.n, 0);
      ti.row0 = __shfl_sync(0xffffffffu, ti.row0, 0);
      ti.rows = __shfl_sync(0xffffffffu, ti.rows, 0);
      ti.kblocks = __shfl_sync(0xffffffffu, ti.kblocks, 0);
      ti.expert = __shfl_sync(0xffffffffu, ti.expert, 0);
      const OpDev* op = &args.ops[ti.kind == kEnd ? args.slots[0] : ti.slot];
      int ok = 1;
      if (lane == 0) {
        // a claimed tile only ever waits on tiles that were claimed before it
        if (ti.kind == kDown) ok = wait_counter(c, &op->g1_done[ti.m], args.I / kTileN1, 3);
        if (ti.kind == kCombine) ok = wait_counter(c, &op->run->gemm_done, op->plan->n_gemm_tiles, 4);
        if (!ok) ti.kind = kEnd;
        fence_async_proxy();
        sc->info[islot] = ti;
        __threadfence_block();
        mbar_arrive(&sc->ifull[islot]);
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (ti.kind == kEnd || !ok) break;
      if (++islot == kRing) { islot = 0; iph ^= 1u; }
      if (ti.kind == kCombine) continue;

      // rows this lane gathers (4 per gather4); rows past the tile's end repeat its last row
      const bool g1 = ti.kind == kGateUp;
      const int n_g = (ti.rows + 3) >> 2;
      int4 idx;
      {
        int r[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int p = ti.row0 + min(4 * lane + i, ti.rows - 1);
          r[i] = g1 ? op->sorted_to_flat[p] / args.k : p;
        }
        idx = make_int4(r[0], r[1], r[2], r[3]);
      }
      const CUtensorMap* tma = g1 ? &op->tm_x : &op->tm_a;
      const CUtensorMap* tmw = g1 ? &op->tm_w1 : &op->tm_w2;
      const int wrow0 = g1 ? ti.expert * 2 * args.I + ti.n * kTileN1 : ti.expert * args.H + ti.n * kTileN2;
      const int wrow1 = g1 ? wrow0 + args.I : wrow0 + 128;
      const unsigned tx = (unsigned)kBBytes + (unsigned)n_g * 512u;
      bool fail = false;
      for (int kb = 0; kb < ti.kblocks; ++kb) {
        if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->empty[stage], ph ^ 1u, 5))) { fail = true; break; }
        unsigned char* sA = stages + (size_t)stage * kStageBytes;
        unsigned char* sB = sA + kABytes;
        if (lane == 0) {
          mbar_expect_tx(&sc->full[stage], tx);
          tma_tile_2d(sB, tmw, kb * kBlockK, wrow0, &sc->full[stage]);
          tma_tile_2d(sB + kBHalfBytes, tmw, kb * kBlockK, wrow1, &sc->full[stage]);
        }
        __syncwarp();
        if (lane < n_g) tma_gather4(sA + lane * 512, tma, kb * kBlockK, idx, &sc->full[stage]);
        if (++stage == kStages) { stage = 0; ph ^= 1u; }
      }
      if (fail) break;
    }
  } else if (warp == 1) {
    // ============================================================ MMA issuer
    int stage = 0, islot = 0, acc = 0;
    unsigned ph = 0, iph = 0, aph[2] = {0, 0};
    while (true) {
      if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->ifull[islot], iph, 6))) break;
      const int kind = sc->info[islot].kind;
      const int kblocks = sc->info[islot].kblocks;
      if (kind == kEnd) break;
      bool fail = false;
      if (kind != kCombine) {
        if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->tempty[acc], aph[acc] ^ 1u, 7))) break;
        tc_fence_after();
        const unsigned d_tmem = tmem + (unsigned)acc * kAccCols;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->full[stage], ph, 8))) { fail = true; break; }
          tc_fence_after();
          if (lane == 0) {
            const unsigned sA = smem_u32(stages + (size_t)stage * kStageBytes);
            const unsigned long long ad = umma_desc(sA), bd = umma_desc(sA + kABytes);
#pragma unroll
            for (int k4 = 0; k4 < kBlockK / 16; ++k4)   // +32 bytes along K per step (>>4 = 2)
              tc_mma_bf16(d_tmem, ad + 2ull * k4, bd + 2ull * k4, kIdesc, (kb | k4) ? 1u : 0u);
            tc_commit(&sc->empty[stage]);               // frees the stage when the MMAs retire
          }
          __syncwarp();
          if (++stage == kStages) { stage = 0; ph ^= 1u; }
        }
        if (fail) break;
        if (lane == 0) tc_commit(&sc->tfull[acc]);       // accumulator complete
        __syncwarp();
        aph[acc] ^= 1u;
        acc ^= 1;
      }
      if (lane == 0) mbar_arrive(&sc->iempty[islot]);
      if (++islot == kRing) { islot = 0; iph ^= 1u; }
    }
  } else {
    // ============================================================ epilogue (warps 2..5)
    const int q = warp & 3;                       // TMEM lane quadrant this warp may read
    const int etid = threadIdx.x - 64;            // 0..127
    int islot = 0, acc = 0;
    unsigned iph = 0, aph[2] = {0, 0};
    while (true) {
      // A failed wait must not leave the other epilogue warps alone at the named barrier
      // below: a warp that gives up records it in shared memory and still joins the barrier;
      // all four warps leave together after it.
      bool ok = __all_sync(0xffffffffu, mbar_wait(c, &sc->ifull[islot], iph, 9));
      TileInfo ti;
      ti.kind = kEnd;
      if (ok) ti = sc->info[islot];
      OpDev* op = &args.ops[ti.kind == kEnd ? args.slots[0] : ti.slot];
      if (ti.kind == kCombine) {
        combine_tokens(op, ti.row0, ti.row0 + ti.rows, args.k, args.H, etid, 128);
      } else if (ti.kind != kEnd) {
        ok = __all_sync(0xffffffffu, mbar_wait(c, &sc->tfull[acc], aph[acc], 10));
        if (ok) {
          tc_fence_after();
          const int row = q * 32 + lane;
          const bool valid = row < ti.rows;
          const unsigned taddr = tmem + (unsigned)acc * kAccCols + ((unsigned)(q * 32) << 16);
          if (q * 32 < ti.rows) {
            if (ti.kind == kGateUp) {
              __nv_bfloat16* dst = op->A + (size_t)(ti.row0 + row) * args.I + ti.n * kTileN1;
#pragma unroll 1
              for (int cch = 0; cch < kTileN1 / 32; ++cch) {
                unsigned g[32], u[32];
                tc_ld32(taddr + cch * 32, g);
                tc_ld32(taddr + 128 + cch * 32, u);
                tc_wait_ld();
                uint4 o[4];
                __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(o);
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                  const float a0 = silu_mul(__uint_as_float(g[2 * i]), __uint_as_float(u[2 * i]));
                  const float a1 = silu_mul(__uint_as_float(g[2 * i + 1]), __uint_as_float(u[2 * i + 1]));
                  oh[i] = __floats2bfloat162_rn(a0, a1);
                }
                if (valid) {
                  uint4* d4 = reinterpret_cast<uint4*>(dst + cch * 32);
#pragma unroll
                  for (int i = 0; i < 4; ++i) d4[i] = o[i];
                }
              }
            } else {
              __nv_bfloat16* dst = op->D + (size_t)(ti.row0 + row) * args.H + ti.n * kTileN2;
#pragma unroll 1
              for (int cch = 0; cch < kTileN2 / 32; ++cch) {
                unsigned v[32];
                tc_ld32(taddr + cch * 32, v);
                tc_wait_ld();
                uint4 o[4];
                __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(o);
#pragma unroll
                for (int i = 0; i < 16; ++i)
                  oh[i] = __floats2bfloat162_rn(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
                if (valid) {
                  uint4* d4 = reinterpret_cast<uint4*>(dst + cch * 32);
#pragma unroll
                  for (int i = 0; i < 4; ++i) d4[i] = o[i];
                }
              }
            }
          }
          tc_fence_before();
          mbar_arrive(&sc->tempty[acc]);          // accumulator may be overwritten
          aph[acc] ^= 1u;
          acc ^= 1;
        }
      }
      if (!ok) *reinterpret_cast<volatile int*>(&sc->epi_fail) = 1;
      __threadfence();
      fence_async_proxy();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (*reinterpret_cast<volatile int*>(&sc->epi_fail) != 0 || ti.kind == kEnd) break;
      if (etid == 0) {
        commit_tile(c, rh, ti);
        mbar_arrive(&sc->iempty[islot]);
      }
      if (++islot == kRing) { islot = 0; iph ^= 1u; }
    }
  }

  // teardown: nothing is claimed any more; let asynchronous work settle, then free TMEM
  if (aborted(c)) __nanosleep(20000);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
  }
}

cudaError_t prepare_run_kernel() {
  return cudaFuncSetAttribute(moe_apk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)kSmemBytes);
}

cudaError_t launch_run(const RunArgs& args, RunHead* rh, int n_ctas, cudaStream_t stream) {
  moe_apk_kernel<<<n_ctas, kThreads, kSmemBytes, stream>>>(args, rh);
  return cudaGetLastError();
}

}  // namespace moe
