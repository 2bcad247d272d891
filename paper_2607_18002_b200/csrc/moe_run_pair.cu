// moe_run on CTA pairs: the bf16 persistent expert kernel with two SMs per tile.
//
// Same scheduling as the single-CTA kernel (two queues, budget word, claim at tile
// boundaries: Sections 4.2 and 6.4), but the unit that claims and runs a tile is a cluster of
// two CTAs on neighbouring SMs, and the MMAs are tcgen05.mma.cta_group::2:
//   - a tile of up to 256 rows runs as ONE M = 256 instruction per k-step: each CTA holds 128
//     of its rows (activations) and 128 of the 256 weight rows of the tile in its own shared
//     memory, the tensor cores of both SMs read both halves of the weight tile.  Per SM that
//     is half the weight bytes through L2 and shared memory for the same flops;
//   - a tile of up to 128 rows runs as M = 128 (64 rows per CTA): the accumulator of a CTA
//     then holds its 64 rows twice, lanes 0..63 against the pair leader's weight rows and
//     lanes 64..127 against the other CTA's;
//   - a stage is 32 KB (16 KB activations + 16 KB weights), six stages deep, and a tile uses
//     256 of the 512 TMEM columns, so the epilogue of one tile overlaps the MMAs of the next.
// Roles per CTA (16 warps): leader only -- warp 0 scheduler (claims, waits for dependencies,
// publishes tile descriptors to both CTAs), warp 1 MMA issuer, warp 2 committer; both CTAs --
// warp 3 producer (TMA loads of its own half, read from the descriptor ring), warps 4-7 gather,
// warps 8-15 epilogue; second CTA only -- warp 1 relays the completion of its gather to the
// leader.  Tile descriptors reach the second CTA through distributed shared memory; its barrier
// arrivals that the leader waits for are remote mbarrier arrivals.  Every wait is bounded, as in
// the single-CTA kernel.
#include "moe_combine.cuh"
#include "moe_ptx.cuh"
#include "moe_sched.cuh"
#include <climits>

namespace moe {
namespace pairk {

constexpr int kThreads = 512;
constexpr int kGatherThreads = 128;
constexpr int kNS = 6;                                   // pipeline stages
constexpr int kABytes = 128 * kRowBytes;                 // up to 128 activation rows of this CTA
constexpr int kBBytes = 128 * kRowBytes;                 // this CTA's 128 weight rows
constexpr int kSB = kABytes + kBBytes;
constexpr int kAccCols = 256;
constexpr int kFullCount = 2 + kGatherThreads + 1;
// instruction descriptors: D fp32, A/B bf16, K-major, N = 256, M = 256 / 128 over the pair
constexpr unsigned kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17);
constexpr unsigned kIdesc256 = kIdescBase | ((256u >> 4) << 24);
constexpr unsigned kIdesc128 = kIdescBase | ((128u >> 4) << 24);

struct SharedCtl {
  alignas(16) TileInfo info[kRing];
  // leader's: everything the MMAs of a stage read is in place.  kFullCount arrivals: one expect_tx
  // per producer (TMA bytes of both CTAs), one per gather thread of the leader (completion of its
  // cp.async copies) and one from the other CTA's relay warp (that CTA's gathered rows are in
  // place); on tiles without a gather the leader's producer arrives in their place
  unsigned long long full[kNS];
  unsigned long long fullA[kNS];     // second CTA: completion of its own gather threads' copies
  unsigned long long goA[kNS];       // producer -> gather warps: the stage may be overwritten
  unsigned long long empty[kNS];     // both (multicast commit): the stage's MMAs retired
  unsigned long long tfull[2];       // both (multicast commit): accumulator complete
  unsigned long long tempty[2];      // leader's: accumulator drained by the 16 epilogue warps
  unsigned long long ifull[kRing];   // own: tile descriptor published
  unsigned long long iempty[kRing];  // leader's: ring slot released by the roles of both CTAs
  unsigned long long done[kRing];    // leader's: the 16 epilogue warps have stored the tile
  unsigned long long taken[kRing];   // leader's: its producer has started on the tile
  unsigned tmem_base;
  alignas(16) unsigned char epi_scratch[8][2048];
  QueueTables qt;
};
static_assert(sizeof(TileInfo) == 48, "descriptor is copied as three 16-byte words");

constexpr size_t kSmemBytes = 1024 + (size_t)kNS * kSB + sizeof(SharedCtl);

// bounded wait that also synchronises with arrivals of the other CTA
__device__ __noinline__ bool wait_slow(const Ctx& c, void* bar, unsigned parity, int where) {
  unsigned long long t0 = 0;
  for (unsigned it = 1;; ++it) {
    if (mbar_try_cluster(bar, parity)) return true;
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
__device__ __forceinline__ bool bwait(const Ctx& c, void* bar, unsigned parity, int where) {
  if (mbar_try_cluster(bar, parity)) return true;
  return wait_slow(c, bar, parity, where);
}
// whole-warp forms.  The cluster-scope wait is for the hand-offs where this thread then reads
// data the other CTA's threads wrote (the tile descriptor, stored outputs); pipeline barriers,
// whose data moves by TMA, tensor core or this CTA's own threads, take the plain wait.
__device__ __forceinline__ bool wwait_cluster(const Ctx& c, void* bar, unsigned parity, int where) {
  return __all_sync(0xffffffffu, bwait(c, bar, parity, where));
}
__device__ __forceinline__ bool wwait(const Ctx& c, void* bar, unsigned parity, int where) {
  return __all_sync(0xffffffffu, mbar_wait(c, bar, parity, where));
}

// A published tile descriptor: in the leader the scheduler's arrival is local, the other CTA reads
// words the leader stored remotely.  The only thing that can delay a descriptor is the scheduler,
// whose own waits are bounded and reported, so this wait gives up later than those (three times
// the limit): a never-ready op is then reported by the wait that met it.
__device__ __noinline__ bool info_wait_one(const Ctx& c, void* bar, unsigned parity, int where, bool leader) {
  unsigned long long t0 = 0;
  for (unsigned it = 1;; ++it) {
    if (leader ? mbar_try(bar, parity) : mbar_try_cluster(bar, parity)) return true;
    if ((it & 63u) == 0) {
      if (aborted(c)) return false;
      const unsigned long long now = gtime_ns();
      if (t0 == 0) t0 = now;
      else if ((long long)(now - t0) > 3 * c.a->wait_ns) {
        report(c.st, MOE_ETIMEOUT, where, (int)blockIdx.x, (int)threadIdx.x, (int)parity);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool wait_info(const Ctx& c, void* bar, unsigned parity, int where, bool leader) {
  return __all_sync(0xffffffffu, info_wait_one(c, bar, parity, where, leader));
}

// arrival on a barrier that lives in the leader's shared memory
__device__ __forceinline__ void arrive_at_leader(void* bar, bool leader) {
  if (leader) mbar_arrive(bar);
  else mbar_arrive_cluster(map_to_cta(bar, 0));
}

// what one CTA loads per k-block of a tile
struct LoadPlan {
  const CUtensorMap* tmw;
  const CUtensorMap* tma;
  int wy0, wy1;       // weight rows of the one or two boxes (wy1 < 0: one box)
  int ay, a_boxes;    // first activation row, number of boxes (0: none or gathered)
  int a_box_rows;
  unsigned tx;
  bool g1;
};

__device__ __forceinline__ LoadPlan make_plan(const RunArgs& a, const OpDev* op, const TileInfo& ti, int rank) {
  LoadPlan p;
  const bool pairT = ti.rows > kTileM;
  const int rpc = pairT ? 128 : 64;
  p.g1 = ti.kind == kGateUp;                 // activation rows come from the gather warps
  const bool w1 = ti.kind != kDown;          // gate/up weights
  p.wy1 = -1;
  p.a_boxes = 0;
  p.a_box_rows = 0;
  p.ay = ti.row0 + rank * rpc;
  p.tma = &op->tm_a8;
  unsigned a_bytes = 0;
  if (w1) {
    const int base = ti.expert * 2 * a.I + ti.n * kTileN1;
    if (pairT) {                 // leader: the 128 gate rows, other CTA: the 128 up rows
      p.tmw = &op->tm_w1;
      p.wy0 = base + (rank ? a.I : 0);
    } else {                     // each CTA: 64 gate rows then the matching 64 up rows
      p.tmw = &op->tm_w1h;
      p.wy0 = base + 64 * rank;
      p.wy1 = base + a.I + 64 * rank;
    }
  } else {
    p.tmw = &op->tm_w2;
    p.wy0 = ti.expert * a.H + ti.n * kTileN2 + 128 * rank;
  }
  if (!p.g1) {
    // consecutive rows: of the packed intermediate (down tile) or of x itself (masked-layout gate/up tile)
    const bool fromx = w1;
    const int mine = min(ti.rows - rank * rpc, rpc);
    if (mine > 0) {
      if (mine <= 8) { p.tma = fromx ? &op->tm_x8 : &op->tm_a8; p.a_boxes = 1; p.a_box_rows = 8; }
      else if (mine <= 32) { p.tma = fromx ? &op->tm_x32 : &op->tm_a32; p.a_boxes = 1; p.a_box_rows = 32; }
      else if (pairT) { p.tma = fromx ? &op->tm_x128 : &op->tm_a128; p.a_boxes = 1; p.a_box_rows = 128; }
      else { p.tma = fromx ? &op->tm_x32 : &op->tm_a32; p.a_boxes = 2; p.a_box_rows = 32; }
      a_bytes = (unsigned)(p.a_boxes * p.a_box_rows * kRowBytes);
    }
  }
  p.tx = (unsigned)kBBytes + a_bytes;
  return p;
}

// one k-block of loads, executed by the whole producer warp with warp-uniform arguments; one
// elected lane issues each instruction (the stage is known to be free)
__device__ __forceinline__ void issue_kblock(SharedCtl* sc, unsigned stages_addr, const LoadPlan& p, int kb,
                                             unsigned stage, bool leader, unsigned full0_addr) {
  const unsigned sA = stages_addr + stage * (unsigned)kSB;
  const unsigned sB = sA + (unsigned)kABytes;
  const unsigned bar = full0_addr + stage * 8u;            // the leader's full[stage]
  // second weight box 64 rows (8 KB) on, second activation box 32 rows (4 KB) and 32 rows on
  static_assert(64 * kRowBytes == 8192 && 32 * kRowBytes == 4096, "offsets used by pair_issue_kblock");
  pair_issue_kblock(bar, p.tx, smem_u32(&sc->full[stage]),
                    (leader && !p.g1) ? (unsigned)kGatherThreads + 1u : 0u,   // nobody gathers for this tile
                    sB, p.tmw, kb * kBlockK, p.wy0, p.wy1, p.wy1 >= 0 ? 1u : 0u,
                    sA, p.tma, p.ay, (unsigned)p.a_boxes,
                    smem_u32(&sc->goA[stage]), p.g1 ? 1u : 0u);
}

// the scheduler hands a tile to the roles of both CTAs
__device__ __forceinline__ void publish(SharedCtl* sc, int islot, const TileInfo& ti) {
  fence_async_proxy();
  sc->info[islot] = ti;
  const unsigned ra = map_to_cta(&sc->info[islot], 1);      // same layout as TileInfo
  st_cluster_v4(ra, make_uint4((unsigned)ti.kind, (unsigned)ti.slot, (unsigned)ti.tile, (unsigned)ti.m));
  st_cluster_v4(ra + 16, make_uint4((unsigned)ti.row0, (unsigned)ti.rows, (unsigned)ti.n, (unsigned)ti.kblocks));
  st_cluster_v4(ra + 32, make_uint4((unsigned)ti.expert, (unsigned)ti.cls, (unsigned)(ti.t_claim & 0xffffffffull),
                                    (unsigned)(ti.t_claim >> 32)));
  mbar_arrive_cluster(map_to_cta(&sc->ifull[islot], 1));   // release: the stores above come first
  __threadfence_block();
  mbar_arrive(&sc->ifull[islot]);
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
moe_apk_pair_kernel(const __grid_constant__ RunArgs args, RunHead* rh) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* stages = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  SharedCtl* sc = reinterpret_cast<SharedCtl*>(stages + (size_t)kNS * kSB);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const bool leader = rank == 0;
  Ctx c{&args, &args.g->status};

  if (threadIdx.x == 0) {
    for (int s = 0; s < kNS; ++s) {
      mbar_init(&sc->full[s], kFullCount);
      mbar_init(&sc->fullA[s], kGatherThreads);
      mbar_init(&sc->goA[s], 1);
      mbar_init(&sc->empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sc->tfull[s], 1);
      mbar_init(&sc->tempty[s], 16);
    }
    // a ring slot is released by: MMA warp, committer, producer, 4 gather warps (leader); producer,
    // relay, 4 gather warps (other CTA)
    for (int s = 0; s < kRing; ++s) {
      mbar_init(&sc->ifull[s], 1);
      mbar_init(&sc->iempty[s], 13);
      mbar_init(&sc->done[s], 16);
      mbar_init(&sc->taken[s], 1);
    }
    if (leader) build_queues(&args, &sc->qt);
    if (blockIdx.x == 0) finish_empty_ops(&args, -1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_proxy();
  }
  if (warp == 1) {   // TMEM of both CTAs (512 columns each); the same warp frees it
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&sc->tmem_base)),
                 "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // the other CTA's barriers exist before anything arrives on them
  tc_fence_after();
  const unsigned tmem = sc->tmem_base;

  if (warp == 0 && leader) {
    // ============================================================ scheduler (leader)
    // Claims a tile, waits (bounded) for a free ring slot, the op's ready word and the tile's
    // dependencies, and publishes it to both CTAs.  The next claim starts when the producer has
    // taken the published tile, so the pair holds at most one claimed tile beyond the one whose
    // loads are being issued.
    int islot = 0;
    unsigned iph = 0;
    TileInfo ti;
    bool need_ready = false;
    ti.kind = kEnd;
    ti.slot = ti.tile = ti.m = ti.row0 = ti.rows = ti.n = ti.kblocks = ti.expert = ti.cls = 0;
    ti.t_claim = 0;
    const bool plain = args.static_kind >= 0;             // plain launch: this pair runs one given entry
    if (plain) claim_static(&args, (int)(blockIdx.x >> 1), ti);
    else claim_next(c, &sc->qt, rh, lane, ti, need_ready);
    while (true) {
      ti.kind = __shfl_sync(0xffffffffu, ti.kind, 0);
      const OpDev* op = &args.ops[ti.kind == kEnd ? args.slots[0] : ti.slot];
      if (!wwait(c, &sc->iempty[islot], iph ^ 1u, 2)) break;
      if (ti.kind != kEnd && need_ready && !wait_op_ready(c, lane, ti)) ti.kind = kEnd;
      int ok = 1;
      if (lane == 0) {
        if (ti.kind == kDown) ok = wait_counter(c, &op->g1_done[ti.m], args.I / kTileN1, 3);
        if (ti.kind == kCombine) ok = wait_counter(c, &op->run->gemm_done, op_gemm_tiles(op), 4);
        if (!ok) ti.kind = kEnd;
        publish(sc, islot, ti);
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      ti.kind = __shfl_sync(0xffffffffu, ti.kind, 0);
      // The gather warps will read the tile's row list (4 bytes per row) first thing: pull it into L2
      // now, the weight stream has usually pushed it out since the plan wrote it.
      if (ti.kind == kGateUp && lane * 32 < ti.rows) prefetch_l2(op->gather_list + ti.row0 + lane * 32);
      if (ti.kind == kEnd || !ok) break;
      if (!wwait(c, &sc->taken[islot], iph, 26)) break;
      if (++islot == kRing) { islot = 0; iph ^= 1u; }
      if (plain) ti.kind = kEnd;
      else claim_next(c, &sc->qt, rh, lane, ti, need_ready);
    }
  } else if (warp == 3) {
    // ============================================================ producer (both CTAs)
    // Reads tiles from the ring and issues this CTA's loads, one stage per k-block.  The whole
    // warp runs the loop on warp-uniform values; one elected lane issues each instruction.
    int islot = 0;
    unsigned iph = 0;
    unsigned stage = 0, par = 1;                           // parity of "stage is free"
    const unsigned stages_addr = smem_u32(stages);
    const unsigned full0_addr = leader ? smem_u32(&sc->full[0]) : map_to_cta(&sc->full[0], 0);
    while (true) {
      if (!wait_info(c, &sc->ifull[islot], iph, 21, leader)) break;
      TileInfo ti;
      ti.kind = __shfl_sync(0xffffffffu, sc->info[islot].kind, 0);
      ti.slot = __shfl_sync(0xffffffffu, sc->info[islot].slot, 0);
      ti.row0 = __shfl_sync(0xffffffffu, sc->info[islot].row0, 0);
      ti.rows = __shfl_sync(0xffffffffu, sc->info[islot].rows, 0);
      ti.n = __shfl_sync(0xffffffffu, sc->info[islot].n, 0);
      ti.kblocks = __shfl_sync(0xffffffffu, sc->info[islot].kblocks, 0);
      ti.expert = __shfl_sync(0xffffffffu, sc->info[islot].expert, 0);
      if (ti.kind == kEnd) break;
      if (lane == 0) {
        arrive_at_leader(&sc->iempty[islot], leader);
        if (leader) mbar_arrive(&sc->taken[islot]);
      }
      if (++islot == kRing) { islot = 0; iph ^= 1u; }
      if (ti.kind == kCombine) continue;
      const LoadPlan lp = make_plan(args, &args.ops[ti.slot], ti, rank);
      bool fail = false;
      for (int kb = 0; kb < ti.kblocks; ++kb) {
        if (!wwait(c, &sc->empty[stage], par, 5)) { fail = true; break; }
        issue_kblock(sc, stages_addr, lp, kb, stage, leader, full0_addr);
        if (++stage == kNS) { stage = 0; par ^= 1u; }
      }
      if (fail) break;
    }
  } else if (warp == 1 && leader) {
    // ============================================================ MMA issuer (leader)
    // The whole warp runs the loops with warp-uniform values and one elected lane issues each
    // MMA and commit: per k-block one barrier wait, four MMAs and one commit, which keeps
    // issuing ahead of the tensor pipe (about 512 clocks per k-block of a 256-row tile).
    int islot = 0;
    unsigned iph = 0, gcount = 0;
    unsigned stage = 0, par = 0;
    const unsigned sbase = smem_u32(stages);
    while (true) {
      if (!wait_info(c, &sc->ifull[islot], iph, 6, true)) break;
      const int kind = __shfl_sync(0xffffffffu, sc->info[islot].kind, 0);
      const int kblocks = __shfl_sync(0xffffffffu, sc->info[islot].kblocks, 0);
      const int rows = __shfl_sync(0xffffffffu, sc->info[islot].rows, 0);
      if (kind == kEnd) break;
      if (kind != kCombine) {
        const unsigned b = gcount & 1u;
        if (!wwait(c, &sc->tempty[b], ((gcount >> 1) & 1u) ^ 1u, 7)) break;
        tc_fence_after();
        const unsigned d = __shfl_sync(0xffffffffu, tmem, 0) + b * (unsigned)kAccCols;
        const unsigned idesc = rows > kTileM ? kIdesc256 : kIdesc128;
        const bool g1 = kind == kGateUp;
        bool fail = false;
        bool ready = false;                           // the current stage was seen full by the look-ahead test
        const unsigned full0 = smem_u32(&sc->full[0]), empty0 = smem_u32(&sc->empty[0]);
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!ready && !wwait(c, &sc->full[stage], par, 8)) { fail = true; break; }
          if (g1) fence_async_proxy_smem();            // this CTA's cp.async-written rows -> tensor core reads
          const unsigned sA = sbase + stage * (unsigned)kSB;
          const unsigned long long ad = umma_desc(sA, kRowBytes), bd = umma_desc(sA + kABytes, kRowBytes);
          const unsigned nstage = stage + 1 == kNS ? 0u : stage + 1, npar = stage + 1 == kNS ? par ^ 1u : par;
          // four MMAs (+32 bytes along K per step: the descriptor's address field counts 16 bytes), the
          // commit that frees the stage in both CTAs, and the test of the next stage's barrier
          ready = pair_mma_kblock(d, ad, bd, idesc, kb ? 1u : 0u, empty0 + stage * 8u, full0 + nstage * 8u, npar);
          ready = __all_sync(0xffffffffu, ready) && kb + 1 < kblocks;
          stage = nstage;
          par = npar;
        }
        if (fail) break;
        tc_commit_pair_elect(&sc->tfull[b]);            // accumulator complete, both CTAs
        ++gcount;
      }
      if (lane == 0) mbar_arrive(&sc->iempty[islot]);
      if (++islot == kRing) { islot = 0; iph ^= 1u; }
    }
  } else if (warp == 1) {
    // ============================================================ gather relay (second CTA)
    // When this CTA's gather threads' copies of a stage have landed it makes them visible to the
    // tensor core (proxy fence) and arrives on the leader's stage barrier.
    int islot = 0;
    unsigned iph = 0, kiter = 0, amask = 0;
    while (true) {
      if (!wait_info(c, &sc->ifull[islot], iph, 24, false)) break;
      const int kind = sc->info[islot].kind;
      const int kblocks = sc->info[islot].kblocks;
      __syncwarp();
      if (kind == kEnd) break;
      if (lane == 0) arrive_at_leader(&sc->iempty[islot], false);
      if (++islot == kRing) { islot = 0; iph ^= 1u; }
      if (kind == kCombine) continue;
      if (kind != kGateUp) { kiter += (unsigned)kblocks; continue; }
      bool fail = false;
      for (int kb = 0; kb < kblocks; ++kb, ++kiter) {
        const int stage = (int)(kiter % kNS);
        if (!wwait(c, &sc->fullA[stage], (amask >> stage) & 1u, 25)) { fail = true; break; }
        amask ^= 1u << stage;
        if (lane == 0) {
          fence_async_proxy_smem();
          mbar_arrive_remote(map_to_cta(&sc->full[stage], 0));
        }
        __syncwarp();
      }
      if (fail) break;
    }
  } else if (warp >= 4 && warp < 4 + kGatherThreads / 32) {
    // ============================================================ gather warps (cp.async)
    // This CTA's rows of a gate/up tile: row r of the tile is token sorted_to_flat[row0 + r] / k.
    // Eight adjacent lanes copy one 128-byte row slice.  Completion is asynchronous: every
    // thread's copies arrive on a barrier when they land (the leader's stage barrier in the
    // leader, a local one that the relay warp forwards in the other CTA), so these warps never
    // wait for their own copies and run as far ahead of the MMAs as the producer does.
    const int gt = threadIdx.x - 128;
    constexpr int kCpr = kRowBytes / 16;                  // 16-byte chunks per row slice
    constexpr int kRowsPerPass = kGatherThreads / kCpr;   // 16 rows per cp.async round
    constexpr int kPasses = 128 / kRowsPerPass;
    const int chunk = gt % kCpr, rbase = gt / kCpr;
    int islot = 0;
    unsigned iph = 0, kiter = 0, gmask = 0;
    while (true) {
      if (!wait_info(c, &sc->ifull[islot], iph, 13, leader)) break;
      const int kind = sc->info[islot].kind;
      const int kblocks = sc->info[islot].kblocks;
      const int rows = sc->info[islot].rows, row0 = sc->info[islot].row0, slot = sc->info[islot].slot;
      __syncwarp();
      if (kind == kEnd) break;
      if (lane == 0) arrive_at_leader(&sc->iempty[islot], leader);
      if (++islot == kRing) { islot = 0; iph ^= 1u; }
      if (kind == kCombine) continue;
      if (kind != kGateUp) { kiter += (unsigned)kblocks; continue; }
      const OpDev* op = &args.ops[slot];
      // a paired op's gather list also holds rows of its partner, tagged with their slot: those come from
      // the partner's activations (kept as the complement of the token index)
      const bool paired = op->paired != 0;
      const OpDev* pop = paired ? &args.ops[op->partner] : op;
      const unsigned char* X = static_cast<const unsigned char*>(op->x) + chunk * 16;
      const unsigned char* Xp = static_cast<const unsigned char*>(pop->x) + chunk * 16;
      const size_t pitch = (size_t)args.H * 2;
      const int rpc = rows > kTileM ? 128 : 64;
      const int first = rank * rpc;                       // this CTA's first row of the tile
      int tok[kPasses];
      const int n_rows = op->n_rows, n_rows_p = pop->n_rows;
      const int own_tag = paired ? slot_of(&args, slot) : 0, partner_tag = paired ? slot_of(&args, op->partner) : 0;
      bool bad = false;
#pragma unroll
      for (int j = 0; j < kPasses; ++j) {
        const int r = rbase + kRowsPerPass * j;
        const bool mine = r < rpc && first + r < rows;
        const int v = mine ? op->gather_list[row0 + first + r] : 0;
        const int tag = v >> kRowSlotShift, flat = v & kRowFlatMask;
        const bool theirs = tag != own_tag;
        // an index the plan never wrote is reported below and its row is skipped
        const bool in_range = v >= 0 && (tag == own_tag || tag == partner_tag) && flat < (theirs ? n_rows_p : n_rows);
        bad |= mine && !in_range;
        tok[j] = (mine && in_range) ? (theirs ? ~(flat / args.k) : flat / args.k) : INT_MIN;
      }
      if (bad) report(c.st, MOE_EBOUNDS, slot_of(&args, slot), row0, rows, 0);
      unsigned long long* landed = leader ? sc->full : sc->fullA;
      bool fail = false;
      for (int kb = 0; kb < kblocks; ++kb, ++kiter) {
        const int stage = (int)(kiter % kNS);
        if (!wwait(c, &sc->goA[stage], (gmask >> stage) & 1u, 14)) { fail = true; break; }
        gmask ^= 1u << stage;
        const unsigned sA = smem_u32(stages + (size_t)stage * kSB);
        const unsigned char* Xk = X + (size_t)kb * kRowBytes;
        const unsigned char* Xpk = Xp + (size_t)kb * kRowBytes;
#pragma unroll
        for (int j = 0; j < kPasses; ++j) {
          const int r = rbase + kRowsPerPass * j;
          const int t = tok[j];
          if (t != INT_MIN)    // the swizzle XORs the chunk index with the row's place in its 8-row group
            cp_async_16(sA + r * kRowBytes + ((chunk ^ (r & 7)) << 4),
                        (t >= 0 ? Xk : Xpk) + (size_t)(t >= 0 ? t : ~t) * pitch);
        }
        cp_async_arrive_noinc(&landed[stage]);
      }
      if (fail) break;
    }
    cp_async_wait_all();
  } else if (warp == 2 && leader) {
    // ============================================================ committer (leader)
    int islot = 0;
    unsigned iph = 0;
    while (true) {
      if (!wait_info(c, &sc->ifull[islot], iph, 16, leader)) break;
      TileInfo ti;
      if (lane == 0) ti = sc->info[islot];
      const int kind = __shfl_sync(0xffffffffu, lane == 0 ? ti.kind : 0, 0);
      if (kind == kEnd) break;
      if (!wwait_cluster(c, &sc->done[islot], iph, 17)) break;
      if (lane == 0) {
        commit_tile(c, rh, ti);
        mbar_arrive(&sc->iempty[islot]);
      }
      __syncwarp();
      if (++islot == kRing) { islot = 0; iph ^= 1u; }
    }
  } else if (warp >= 8) {
    // ============================================================ epilogue (8 warps per CTA)
    // Warp w reads TMEM lanes 32 (w % 4) .. +31.  M = 256 tiles: lane = one of this CTA's 128
    // rows, 256 columns.  M = 128 tiles: lanes 0..63 and 64..127 both hold this CTA's 64
    // rows, against the first / second 128 weight rows of the tile (128 columns).
    const int q = warp & 3;
    const int half = (warp - 8) >> 2;             // the two warps of a quadrant split the columns
    const int etid = threadIdx.x - 256;
    int islot = 0;
    unsigned iph = 0, gcount = 0;
    unsigned char* scratch = sc->epi_scratch[warp - 8];
    const int srow = lane >> 2, schunk = lane & 3;
    while (true) {
      if (!wait_info(c, &sc->ifull[islot], iph, 9, leader)) break;
      const TileInfo ti = sc->info[islot];
      if (ti.kind == kEnd) break;
      OpDev* op = &args.ops[ti.slot];
      bool ok = true;
      if (ti.kind == kCombine) {
        const int mid = ti.row0 + (ti.rows + 1) / 2;
        if (leader) combine_tokens(op, ti.row0, mid, args.k, args.H, etid, 256);
        else combine_tokens(op, mid, ti.row0 + ti.rows, args.k, args.H, etid, 256);
      } else {
        const int b = (int)(gcount & 1u);
        ok = wwait(c, &sc->tfull[b], (gcount >> 1) & 1u, 10);
        if (!ok) break;
        ++gcount;
        tc_fence_after();
        const bool pairT = ti.rows > kTileM;
        const bool g1 = ti.kind != kDown;                     // gate/up tile: SwiGLU, output to A
        const int rpc = pairT ? 128 : 64;
        const int lrow0 = pairT ? q * 32 : (q & 1) * 32;     // first of this warp's rows within the CTA's rows
        const int cg = pairT ? 0 : (q >> 1);                  // which 128 weight rows (M = 128 tiles)
        const int ncols = pairT ? (g1 ? 128 : 256) : (g1 ? 64 : 128);   // output columns held per lane
        const int upoff = pairT ? 128 : 64;                   // column distance gate -> up
        const int passes = ncols / 64;                        // 32-column passes per warp
        const int trow0 = rank * rpc + lrow0;                 // tile row of lane 0
        const int rows_here = min(32, ti.rows - trow0);
        const size_t pitch = (size_t)(g1 ? args.I : args.H) * 2;
        if (rows_here > 0) {
          const unsigned taddr = tmem + (unsigned)(b * kAccCols) + ((unsigned)(q * 32) << 16);
          unsigned char* out = reinterpret_cast<unsigned char*>(g1 ? (void*)op->A : (void*)op->D) +
                               (size_t)(ti.row0 + trow0) * pitch +
                               ((size_t)ti.n * (g1 ? kTileN1 : kTileN2) + (size_t)cg * ncols) * 2;
          unsigned g[32], u[32];
          tc_ld32(taddr + (half * passes) * 32, g);
          if (g1) tc_ld32(taddr + upoff + (half * passes) * 32, u);
#pragma unroll 1
          for (int p = 0; p < passes; ++p) {
            const int pass = half * passes + p;
            uint4 o[4];
            __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(o);
            tc_wait_ld();
            if (g1) {
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                const float a0 = silu_mul(__uint_as_float(g[2 * i]), __uint_as_float(u[2 * i]));
                const float a1 = silu_mul(__uint_as_float(g[2 * i + 1]), __uint_as_float(u[2 * i + 1]));
                oh[i] = __floats2bfloat162_rn(a0, a1);
              }
            } else {
#pragma unroll
              for (int i = 0; i < 16; ++i)
                oh[i] = __floats2bfloat162_rn(__uint_as_float(g[2 * i]), __uint_as_float(g[2 * i + 1]));
            }
            if (p + 1 < passes) {
              tc_ld32(taddr + (pass + 1) * 32, g);
              if (g1) tc_ld32(taddr + upoff + (pass + 1) * 32, u);
            }
            __syncwarp();                                          // scratch free again
#pragma unroll
            for (int j = 0; j < 4; ++j)     // row `lane`, 16-byte chunk j (XOR keeps banks apart)
              *reinterpret_cast<uint4*>(scratch + lane * 64 + ((j ^ ((lane >> 1) & 3)) << 4)) = o[j];
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int r = 8 * j + srow;
              const uint4 v4 = *reinterpret_cast<const uint4*>(scratch + r * 64 + ((schunk ^ ((r >> 1) & 3)) << 4));
              if (r < rows_here)
                *reinterpret_cast<uint4*>(out + (size_t)r * pitch + pass * 64 + schunk * 16) = v4;
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) arrive_at_leader(&sc->tempty[b], leader);   // accumulator may be overwritten
      }
      __syncwarp();
      if (lane == 0) {
        __threadfence();                          // the warp's stores, before the tile is published
        arrive_at_leader(&sc->done[islot], leader);
      }
      if (++islot == kRing) { islot = 0; iph ^= 1u; }
    }
  }

  // teardown: nothing is claimed any more; let asynchronous work settle, then free TMEM
  if (aborted(c)) __nanosleep(20000);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // no CTA leaves while the other may still signal its barriers
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
  }
}

}  // namespace pairk

cudaError_t prepare_pair_kernel() {
  return cudaFuncSetAttribute(pairk::moe_apk_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)pairk::kSmemBytes);
}

// n_ctas: the persistent grid, or 2 x the number of queue entries for a plain launch
cudaError_t launch_pair(const RunArgs& args, RunHead* rh, int n_ctas, cudaStream_t stream) {
  pairk::moe_apk_pair_kernel<<<n_ctas, pairk::kThreads, pairk::kSmemBytes, stream>>>(args, rh);
  return cudaGetLastError();
}

}  // namespace moe
