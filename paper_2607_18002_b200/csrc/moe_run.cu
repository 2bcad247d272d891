// moe_run: the persistent expert kernel (the adaptive persistent kernel of Section 4 of the
// paper, rebuilt for sm_100a), one CTA per tile.  This kernel runs the FP8 e4m3 path, and bf16 on
// grids with an odd number of CTAs; bf16 on an even grid runs on CTA pairs (moe_run_pair.cu).
//
// One CTA per SM, 16 warps with fixed roles:
//   warp 0      scheduler + producer.  At every tile boundary it reads the decode budget
//               word and the two queue heads, claims the next tile (decode first for CTAs
//               below the budget, prefill first for the others, each falling back to the
//               other class: Sections 4.2 and 6.4), hands the tile to the other warps
//               through a shared-memory ring guarded by mbarriers (the hand-off of
//               Section 4.3: the first pipeline warp decides, later warps follow), waits for
//               the tile's dependencies, then feeds the pipeline: weight tiles (and the
//               packed intermediate rows of a down tile) by tiled TMA.
//   warp 1      issues tcgen05.mma (128 x 256 x 16, bf16 -> fp32) into the TMEM accumulators;
//               tcgen05.commit releases pipeline stages and publishes the accumulators.  A
//               tile of up to 256 rows runs as two 128-row MMAs per k-step against the SAME
//               weight tile in shared memory, which halves the weight bytes moved per flop.
//   warp 2      committer: when the epilogue threads have stored a tile it fences and bumps the
//               dependency counters, the op's done word and the tile log.
//   warp 3      idle (it only joins the final barrier).
//   warps 4-7   gather: the activation rows of a gate/up tile are scattered tokens; they are
//               copied through the permutation with 16-byte cp.async into the swizzled
//               layout the tensor core reads.
//   warps 8-15  epilogue: tcgen05.ld, SwiGLU (gate/up tiles), bf16 stores transposed through
//               shared memory into row segments.  They also run the combine tiles.
// A phase switch happens only between tiles, so no accumulator, TMA transaction or buffer is
// live across it (Section 4.2) and results are independent of the schedule.
//
// Every wait (mbarrier, dependency counter, ready word) is bounded: when it runs out the
// kernel records MOE_ETIMEOUT, raises the abort word, and all CTAs drain and return.
#include "moe_combine.cuh"
#include "moe_ptx.cuh"
#include "moe_sched.cuh"
#include <cuda_fp8.h>
#include <climits>

namespace moe {

constexpr int kGatherThreads = 128;                     // 4 gather warps
constexpr int kThreads = 512;                           // 16 warps, see the role list above
constexpr int kAHalfBytes = kTileM * kRowBytes;        // 128 activation rows of one k-block
constexpr int kABytes = 2 * kAHalfBytes;               // up to 256 activation rows per stage
constexpr int kBHalfBytes = 128 * kRowBytes;           // 128 weight rows of one k-block
constexpr int kBBytes = 2 * kBHalfBytes;               // 256 weight rows per stage
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kMaxStages = 4;                          // fp8: four 48 KB stages, bf16: three 64 KB stages
constexpr int kAccCols = 256;                          // TMEM columns per accumulator

struct SharedCtl {
  unsigned long long full[kMaxStages], fullA[kMaxStages], empty[kMaxStages];
  unsigned long long tfull[2], tempty[2];
  unsigned long long pfull[2], pempty[2];          // fp8: per-k-block partial products, two 256-column buffers
  unsigned long long xbar[4];                      // fp8: amax exchange between the two warps of a quadrant
  float amax_x[2][4][32];
  unsigned long long ifull[kRing], iempty[kRing], done[kRing];
  TileInfo info[kRing];
  unsigned tmem_base;
  alignas(16) unsigned char epi_scratch[8][2048];   // per epilogue warp: 32 rows x 64 bytes
  QueueTables qt;
};

constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + sizeof(SharedCtl);

// ------------------------------------------------------------------ FP8 (e4m3, fp32 block scales)
// instruction descriptor: D fp32, A/B e4m3, both K-major, M = 128, N = 256
constexpr unsigned kIdescF8 = (1u << 4) | ((256u >> 3) << 17) | ((128u >> 4) << 24);

// One e4m3 tile on the epilogue warps.  Thread = (accumulator row, 64-column slice of each
// 128-column half); its 128 fp32 accumulators stay in registers (the epilogue warps raise
// their register allowance for this).  Per k-block and half: partial * (activation scale of
// the row and k-block * weight scale of the half and k-block) is added in.  Then gate/up
// tiles apply SwiGLU and re-quantise the 128 outputs of the row to e4m3 with one fp32 scale
// (amax / 448) -- the one quantisation on the path -- and down tiles store bf16.
__device__ __forceinline__ bool epilogue_fp8(const Ctx& c, SharedCtl* sc, OpDev* op, const TileInfo& ti,
                                             unsigned tmem, int warp, int lane, unsigned& eph,
                                             unsigned& xph) {
  const RunArgs& a = *c.a;
  const int q = warp & 3, ch = (warp - 8) >> 2;
  const int row = q * 32 + lane;
  const bool valid = row < ti.rows;
  const bool g1 = ti.kind != kDown;
  const int HB = a.H / 128, IB = a.I / 128;
  const unsigned lane_addr = tmem + ((unsigned)(q * 32) << 16);
  // scale streams of this row / tile
  const float* sx;
  const float *sw0, *sw1;
  if (ti.kind == kGateUpDirect) {       // masked layout: the row's scales sit at the row's own index
    sx = op->x_scale + (size_t)(ti.row0 + (valid ? row : 0)) * HB;
    sw0 = op->s_gate_up + ((size_t)ti.expert * (2 * IB) + ti.n) * HB;
    sw1 = op->s_gate_up + ((size_t)ti.expert * (2 * IB) + IB + ti.n) * HB;
  } else if (g1) {
    // the row's activation scales: its own op's, or (paired form) the partner's when the row is tagged so
    int tok = 0;
    const OpDev* src = op;
    if (valid) {
      const int v = op->gather_list[ti.row0 + row];
      const int tag = v >> kRowSlotShift, flat = v & kRowFlatMask;
      const int own_tag = op->paired ? slot_of(&a, ti.slot) : 0;
      if (op->paired && tag != own_tag && tag == slot_of(&a, op->partner)) src = &a.ops[op->partner];
      if (v >= 0 && (tag == own_tag || src != op) && flat < src->n_rows) tok = flat / a.k;
      else { src = op; report(c.st, MOE_EBOUNDS, slot_of(&a, ti.slot), ti.row0 + row, v, 1); }
    }
    sx = src->x_scale + (size_t)tok * HB;
    sw0 = op->s_gate_up + ((size_t)ti.expert * (2 * IB) + ti.n) * HB;
    sw1 = op->s_gate_up + ((size_t)ti.expert * (2 * IB) + IB + ti.n) * HB;
  } else {
    sx = op->a_scale + (size_t)(ti.row0 + (valid ? row : 0)) * IB;
    sw0 = op->s_down + ((size_t)ti.expert * HB + 2 * ti.n) * IB;
    sw1 = sw0 + IB;
  }
  if (q * 32 >= ti.rows) {
    // No row of the tile lies in this warp's TMEM lane quadrant (both warps of a quadrant see
    // the same q): nothing to read, scale or store.  The warp still takes part in every partial
    // buffer hand-off, so that the barrier counts and phases stay those of a full tile.
    for (int kb = 0; kb < ti.kblocks; ++kb) {
      const int pb = kb & 1;
      if (!__all_sync(0xffffffffu, mbar_wait_inline(c, &sc->pfull[pb], (eph >> pb) & 1u, 19))) return false;
      eph ^= 1u << pb;
      if (lane == 0) mbar_arrive(&sc->pempty[pb]);
    }
    return true;
  }
  float acc[128];                                 // [half][64]
#pragma unroll
  for (int i = 0; i < 128; ++i) acc[i] = 0.f;
  // scales of the next k-block are loaded one k-block ahead (three scalars in flight)
  float nfx = 0.f, nw0 = 0.f, nw1 = 0.f;
  if (ti.kblocks > 0) { nfx = sx[0]; nw0 = sw0[0]; nw1 = sw1[0]; }
  for (int kb = 0; kb < ti.kblocks; ++kb) {
    const float s0 = nfx * nw0, s1 = nfx * nw1;
    if (kb + 1 < ti.kblocks) { nfx = sx[kb + 1]; nw0 = sw0[kb + 1]; nw1 = sw1[kb + 1]; }
    const int pb = kb & 1;
    if (!__all_sync(0xffffffffu, mbar_wait_inline(c, &sc->pfull[pb], (eph >> pb) & 1u, 19))) return false;
    eph ^= 1u << pb;
    tc_fence_after();
    // four 32-column chunks (two per half), one TMEM load each: tcgen05.wait::ld waits for every load of the
    // thread, so a second load in flight only ever overlapped one chunk's FMAs; fewer, wider loads are faster
    // (the other warp of the scheduler partition fills the wait)
    const unsigned pbase = lane_addr + (unsigned)(pb * 256 + ch * 64);
    unsigned p[32];
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
      tc_ld32(pbase + (unsigned)((cc >> 1) * 128 + (cc & 1) * 32), p);
      tc_wait_ld();
      const float s = (cc >> 1) ? s1 : s0;
#pragma unroll
      for (int i = 0; i < 32; ++i)
        acc[cc * 32 + i] = fmaf(__uint_as_float(p[i]), s, acc[cc * 32 + i]);
    }
    tc_fence_before();
    __syncwarp();                                 // every lane's TMEM loads have completed
    if (lane == 0) mbar_arrive(&sc->pempty[pb]); // one arrival per warp: the partial buffer may be overwritten
  }
  // the accumulator is complete
  if (g1) {
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < 64; ++i) {                // gate column i and up column i of this slice
      const float gv = acc[i];
      const float v = __fdividef(gv, 1.0f + __expf(-gv)) * acc[64 + i];
      acc[i] = v;
      amax = fmaxf(amax, fabsf(v));
    }
    // the row's 128 outputs live in two threads (ch = 0, 1): exchange the partial maxima
    sc->amax_x[ch][q][lane] = amax;
    mbar_arrive(&sc->xbar[q]);
    if (!__all_sync(0xffffffffu, mbar_wait_inline(c, &sc->xbar[q], xph, 20))) return false;
    xph ^= 1u;
    amax = fmaxf(amax, sc->amax_x[ch ^ 1][q][lane]);
    const float scale = amax > 0.f ? amax / 448.0f : 1.0f;
    const float inv = amax > 0.f ? 448.0f / amax : 0.0f;
    if (valid) {
      unsigned char* dst = static_cast<unsigned char*>((void*)op->A) + (size_t)(ti.row0 + row) * a.I +
                           (size_t)ti.n * 128 + ch * 64;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        unsigned w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int b0 = j * 16 + i * 4;
          const unsigned lo = __nv_cvt_float2_to_fp8x2(make_float2(acc[b0] * inv, acc[b0 + 1] * inv), __NV_SATFINITE, __NV_E4M3);
          const unsigned hi = __nv_cvt_float2_to_fp8x2(make_float2(acc[b0 + 2] * inv, acc[b0 + 3] * inv), __NV_SATFINITE, __NV_E4M3);
          w[i] = lo | (hi << 16);
        }
        reinterpret_cast<uint4*>(dst)[j] = make_uint4(w[0], w[1], w[2], w[3]);
      }
      if (ch == 0) op->a_scale[(size_t)(ti.row0 + row) * IB + ti.n] = scale;
    }
  } else if (valid) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      __nv_bfloat16* dst = op->D + (size_t)(ti.row0 + row) * a.H + (size_t)ti.n * kTileN2 + h * 128 + ch * 64;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        uint4 o4;
        __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&o4);
#pragma unroll
        for (int i = 0; i < 4; ++i)
          oh[i] = __floats2bfloat162_rn(acc[h * 64 + j * 8 + 2 * i], acc[h * 64 + j * 8 + 2 * i + 1]);
        reinterpret_cast<uint4*>(dst)[j] = o4;
      }
    }
  }
  return true;
}

// ------------------------------------------------------------------ the persistent kernel
// which accumulator(s) a tile uses: a tile of up to 128 rows alternates between the two, a
// tile of up to 256 rows takes both (rows 0..127 -> accumulator 0, rows 128..255 -> 1).
// Every role walks the same tile sequence, so each derives this locally.
struct AccUse {
  int next = 0;
  __device__ __forceinline__ void take(int rows, bool& use0, bool& use1) {
    if (rows > kTileM) { use0 = use1 = true; }
    else { use0 = next == 0; use1 = !use0; next ^= 1; }
  }
};

template <bool kFp8>
__global__ void __launch_bounds__(kThreads, 1) moe_apk_kernel(const __grid_constant__ RunArgs args,
                                                              RunHead* rh) {
  constexpr int kKb = kFp8 ? 128 : kBlockK;     // K elements per stage (128 bytes per row either way)
  constexpr int kEl = kFp8 ? 1 : 2;             // bytes per element
  // fp8 tiles have at most 128 rows: a stage holds 128 activation rows + 256 weight rows
  constexpr int kNS = kFp8 ? 4 : 3;
  constexpr int kBOff = kFp8 ? kAHalfBytes : kABytes;
  constexpr int kSB = kBOff + kBBytes;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* stages = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  SharedCtl* sc = reinterpret_cast<SharedCtl*>(stages + (size_t)kNS * kSB);
  static_assert(kNS * kSB == 3 * (kABytes + kBBytes), "ring size");
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  Ctx c{&args, &args.g->status};

  if (threadIdx.x == 0) {
    for (int s = 0; s < kNS; ++s) {
      mbar_init(&sc->full[s], 1);
      mbar_init(&sc->fullA[s], kGatherThreads);
      mbar_init(&sc->empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sc->tfull[s], 1);
      mbar_init(&sc->tempty[s], 256);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sc->pfull[s], 1);
      mbar_init(&sc->pempty[s], 8);
    }
    for (int s = 0; s < 4; ++s) mbar_init(&sc->xbar[s], 64);
    // a ring slot is released by the MMA warp, the committer and each gather warp
    for (int s = 0; s < kRing; ++s) {
      mbar_init(&sc->ifull[s], 1);
      mbar_init(&sc->iempty[s], 2 + kGatherThreads / 32);
      mbar_init(&sc->done[s], 256);
    }
    build_queues(&args, &sc->qt);
    if (blockIdx.x == 0) finish_empty_ops(&args, -1);
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
  // The fp8 epilogue keeps 128 fp32 accumulators per thread: the two epilogue warpgroups take
  // registers from the two others (64 + 192 = 2 x 128 per thread pair).  Each role changes its
  // allowance at the top of its own branch, so the compiler can budget the branch by it.
#define MOE_REGS_DEC() do { if constexpr (kFp8) asm volatile("setmaxnreg.dec.sync.aligned.u32 64;"); } while (0)
#define MOE_REGS_INC() do { if constexpr (kFp8) asm volatile("setmaxnreg.inc.sync.aligned.u32 192;"); } while (0)

  if (warp == 0) {
    MOE_REGS_DEC();
    // ============================================================ scheduler + TMA producer
    // The next tile is claimed while the current one is still being loaded (after its
    // kClaimAt-th k-block), so the claim's round trips and the first loads of the next tile
    // overlap the current tile's tail instead of draining the pipeline.  A CTA therefore
    // holds at most one claimed tile beyond the one it is executing.
    int stage = 0, islot = 0;
    unsigned ph = 0, iph = 0;
    TileInfo ti, nx;
    bool ti_need_ready = false, nx_need_ready = false, have_nx = false;
    bool ti_published = false, nx_published = false;
    ti.kind = kEnd;
    ti.slot = ti.tile = ti.m = ti.row0 = ti.rows = ti.n = ti.kblocks = ti.expert = ti.cls = 0;
    ti.t_claim = 0;
    nx = ti;
    claim_next(c, &sc->qt, rh, lane, ti, ti_need_ready);
    while (true) {
      ti.kind = __shfl_sync(0xffffffffu, ti.kind, 0);      // the claim loops exit warp-uniformly
      const OpDev* op = &args.ops[ti.kind == kEnd ? args.slots[0] : ti.slot];
      if (!ti_published) {
        // blocking hand-off: a free ring slot, the op ready, the tile's dependencies met
        if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->iempty[islot], iph ^ 1u, 2))) break;
        if (ti.kind != kEnd && ti_need_ready && !wait_op_ready(c, lane, ti)) ti.kind = kEnd;
        int ok = 1;
        if (lane == 0) {
          // a claimed tile only ever waits on tiles that were claimed before it
          if (ti.kind == kDown) ok = wait_counter(c, &op->g1_done[ti.m], args.I / kTileN1, 3);
          if (ti.kind == kCombine) ok = wait_counter(c, &op->run->gemm_done, op_gemm_tiles(op), 4);
          if (!ok) ti.kind = kEnd;
          fence_async_proxy();
          sc->info[islot] = ti;
          __threadfence_block();
          mbar_arrive(&sc->ifull[islot]);
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (ti.kind == kEnd || !ok) break;
        if (++islot == kRing) { islot = 0; iph ^= 1u; }
      }
      ti_published = false;

      if (ti.kind != kCombine) {
        // Weight tiles by tiled TMA.  The A operand of a down tile is the packed intermediate:
        // consecutive rows, one TMA box (8, 32, 128 or 256 rows high, the smallest that holds
        // the tile's rows); the A operand of a gate/up tile is gathered by the gather warps.
        const bool g1 = ti.kind != kDown;                  // gate/up weights
        const bool gathered = ti.kind == kGateUp;          // activation rows come from the gather warps
        const bool fromx = ti.kind == kGateUpDirect;       // ... or are consecutive rows of x (masked layout)
        const CUtensorMap* tmw = g1 ? &op->tm_w1 : &op->tm_w2;
        const int wrow0 = g1 ? ti.expert * 2 * args.I + ti.n * kTileN1 : ti.expert * args.H + ti.n * kTileN2;
        const int wrow1 = g1 ? wrow0 + args.I : wrow0 + 128;
        const int box = ti.rows <= 8 ? 8 : (ti.rows <= 32 ? 32 : (ti.rows <= 128 ? 128 : 256));
        const CUtensorMap* tma = fromx ? (box == 8 ? &op->tm_x8 : (box == 32 ? &op->tm_x32 : (box == 128 ? &op->tm_x128 : &op->tm_x256)))
                                       : (box == 8 ? &op->tm_a8 : (box == 32 ? &op->tm_a32 : (box == 128 ? &op->tm_a128 : &op->tm_a256)));
        const unsigned tx = (unsigned)kBBytes + (gathered ? 0u : (unsigned)(box * kRowBytes));
        const int claim_at = min(kClaimAt, ti.kblocks - 1);
        bool fail = false;
        for (int kb = 0; kb < ti.kblocks; ++kb) {
          if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->empty[stage], ph ^ 1u, 5))) { fail = true; break; }
          {
            const unsigned sA = smem_u32(stages + (size_t)stage * kSB);
            single_issue_kblock(smem_u32(&sc->full[stage]), tx, sA + kBOff, sA + kBOff + kBHalfBytes, tmw, kb * kKb,
                                wrow0, wrow1, sA, tma, ti.row0, gathered ? 0u : 1u);
          }
          if (++stage == kNS) { stage = 0; ph ^= 1u; }
          if (kb == claim_at)              // claim ahead (never blocks here)
            have_nx = claim_once(c, &sc->qt, rh, lane, nx, nx_need_ready) == 1;
          if (have_nx && !nx_published && kb > claim_at && kb >= ti.kblocks - kPublishLead) {
            // Hand the next tile to the other warps before this one's last loads go out, if that
            // takes no waiting: free ring slot, op ready, dependencies already met.
            const OpDev* nop = &args.ops[nx.slot];
            bool can = __all_sync(0xffffffffu, mbar_try(&sc->iempty[islot], iph ^ 1u));
            if (can && nx_need_ready) can = __shfl_sync(0xffffffffu, op_ready(&args, nop) ? 1 : 0, 0) != 0;   // lane 0's look
            if (can) {
              int met = 1;
              if (lane == 0) {
                if (nx.kind == kDown) met = ld_acquire(&nop->g1_done[nx.m]) >= args.I / kTileN1;
                if (nx.kind == kCombine) met = ld_acquire(&nop->run->gemm_done) >= op_gemm_tiles(nop);
                if (met) {
                  fence_async_proxy();
                  sc->info[islot] = nx;
                  __threadfence_block();
                  mbar_arrive(&sc->ifull[islot]);
                }
              }
              met = __shfl_sync(0xffffffffu, met, 0);
              if (met) {
                nx_published = true;
                if (++islot == kRing) { islot = 0; iph ^= 1u; }
              }
            }
          }
        }
        if (fail) break;
      }
      if (have_nx) {
        ti = nx;
        ti_need_ready = nx_need_ready;
        ti_published = nx_published;
        have_nx = nx_published = false;
      } else {
        claim_next(c, &sc->qt, rh, lane, ti, ti_need_ready);
      }
    }
  } else if (warp == 1) {
    MOE_REGS_DEC();
    // ============================================================ MMA issuer
    int stage = 0, islot = 0;
    unsigned ph = 0, iph = 0, aph[2] = {0, 0}, pph = 0;
    AccUse accs;
    while (true) {
      if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->ifull[islot], iph, 6))) break;
      const int kind = sc->info[islot].kind;
      const int kblocks = sc->info[islot].kblocks;
      const int rows = sc->info[islot].rows;
      if (kind == kEnd) break;
      bool fail = false;
      if (kFp8 && kind != kCombine) {
        // FP8 with fp32 block scales: the tensor core cannot apply a scale per 128-deep K block,
        // so every k-block (= one scale block) is multiplied into a FRESH partial buffer, one
        // per 128-column half of the weight tile (each half has a single weight scale), and the
        // epilogue warps scale-and-add it into the fp32 accumulator columns of TMEM.
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->full[stage], ph, 8))) { fail = true; break; }
          if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->fullA[stage], ph, 12))) { fail = true; break; }
          {
            const int pb = kb & 1;                        // partial buffer of this k-block
            if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->pempty[pb], ((pph >> pb) & 1u) ^ 1u, 18))) { fail = true; break; }
            pph ^= 1u << pb;
            tc_fence_after();
            {
              fence_async_proxy_smem();
              const unsigned sA = smem_u32(stages + (size_t)stage * kSB);
              const unsigned long long ad = umma_desc(sA, kRowBytes);
              const unsigned long long bd = umma_desc(sA + kBOff, kRowBytes);
              // four MMAs of 32 e4m3 elements (32 bytes) each, partial full, stage empty
              f8_mma_kblock(tmem + (unsigned)(pb * 256), ad, bd, kIdescF8, smem_u32(&sc->pfull[pb]),
                            smem_u32(&sc->empty[stage]));
            }
          }
          if (fail) break;
          if (++stage == kNS) { stage = 0; ph ^= 1u; }
        }
        if (fail) break;
      } else if (kind != kCombine) {
        bool use0, use1;
        accs.take(rows, use0, use1);
        // A 256-row tile takes both accumulators: it waits for accumulator 1 only when its first
        // MMA into it is due, so the drain of accumulator 1 overlaps the tile's first MMAs.
        const bool pair = use0 && use1;
        if (use0 && !__all_sync(0xffffffffu, mbar_wait(c, &sc->tempty[0], aph[0] ^ 1u, 7))) break;
        if (use1 && !pair && !__all_sync(0xffffffffu, mbar_wait(c, &sc->tempty[1], aph[1] ^ 1u, 7))) break;
        tc_fence_after();
        const unsigned d0 = tmem + (use0 ? 0u : (unsigned)kAccCols);     // accumulator of rows 0..127
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->full[stage], ph, 8))) { fail = true; break; }
          // The gather warps arrive on fullA for every k-block (with the copied rows of a
          // gate/up tile, empty-handed otherwise): being part of every stage hand-off keeps them
          // within one phase of the stage barriers they wait on.
          if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->fullA[stage], ph, 12))) { fail = true; break; }
          tc_fence_after();
          if (lane == 0) {
            fence_async_proxy_smem();                    // cp.async-written rows -> tensor core reads
            const unsigned sA = smem_u32(stages + (size_t)stage * kSB);
            const unsigned long long ad = umma_desc(sA, kRowBytes), bd = umma_desc(sA + kBOff, kRowBytes);
#pragma unroll
            for (int k4 = 0; k4 < kBlockK / 16; ++k4)   // +32 bytes along K per step (>>4 = 2)
              tc_mma_bf16(d0, ad + 2ull * k4, bd + 2ull * k4, kIdesc, (kb | k4) ? 1u : 0u);
          }
          if (pair && kb == 0) {                         // accumulator 1 is needed from here on
            if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->tempty[1], aph[1] ^ 1u, 7))) { fail = true; break; }
            tc_fence_after();
          }
          if (lane == 0) {
            const unsigned sA = smem_u32(stages + (size_t)stage * kSB);
            const unsigned long long bd = umma_desc(sA + kBOff, kRowBytes);
            if (pair) {                                  // rows 128..255 against the same weight tile
              const unsigned long long ad1 = umma_desc(sA + kAHalfBytes, kRowBytes);
#pragma unroll
              for (int k4 = 0; k4 < kBlockK / 16; ++k4)
                tc_mma_bf16(tmem + (unsigned)kAccCols, ad1 + 2ull * k4, bd + 2ull * k4, kIdesc, (kb | k4) ? 1u : 0u);
            }
            tc_commit(&sc->empty[stage]);               // frees the stage when the MMAs retire
          }
          __syncwarp();
          if (++stage == kNS) { stage = 0; ph ^= 1u; }
        }
        if (fail) break;
        if (lane == 0) {                                 // accumulator(s) complete
          if (use0) tc_commit(&sc->tfull[0]);
          if (use1) tc_commit(&sc->tfull[1]);
        }
        __syncwarp();
        if (use0) aph[0] ^= 1u;
        if (use1) aph[1] ^= 1u;
      }
      if (lane == 0) mbar_arrive(&sc->iempty[islot]);
      if (++islot == kRing) { islot = 0; iph ^= 1u; }
    }
  } else if (warp >= 4 && warp < 4 + kGatherThreads / 32) {
    MOE_REGS_DEC();
    // ============================================================ gather warps (cp.async)
    // Rows of a gate/up tile are scattered tokens: row r of the tile is token
    // sorted_to_flat[row0 + r] / k.  Adjacent lanes copy one row slice (16 bytes each)
    // into the swizzled layout the tensor core reads.
    const int gt = threadIdx.x - 128;
    constexpr int kCpr = kRowBytes / 16;                  // 16-byte chunks per row slice
    constexpr int kRowsPerPass = kGatherThreads / kCpr;   // rows covered by one cp.async per thread
    constexpr int kPasses = (kFp8 ? 128 : 256) / kRowsPerPass;   // fp8 work tiles have at most 128 rows
    const int chunk = gt % kCpr, rbase = gt / kCpr;       // rows rbase + kRowsPerPass * j
    int islot = 0;
    unsigned iph = 0, kiter = 0;                          // kiter: k-blocks of all GEMM tiles so far
    while (true) {
      if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->ifull[islot], iph, 13))) break;
      const int kind = sc->info[islot].kind;
      const int kblocks = sc->info[islot].kblocks;
      const int rows = sc->info[islot].rows, row0 = sc->info[islot].row0, slot = sc->info[islot].slot;
      __syncwarp();
      if (lane == 0) mbar_arrive(&sc->iempty[islot]);
      if (++islot == kRing) { islot = 0; iph ^= 1u; }
      if (kind == kEnd) break;
      if (kind == kCombine) continue;
      if (kind != kGateUp) {           // nothing to gather: hand every stage on empty-handed
        bool failed = false;
        for (int kb = 0; kb < kblocks; ++kb, ++kiter) {
          const int stage = (int)(kiter % kNS);
          if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->empty[stage], ((kiter / kNS) & 1u) ^ 1u, 15))) { failed = true; break; }
          if (lane == 0) mbar_arrive_n(&sc->fullA[stage], 32);   // the whole warp's share in one arrival
        }
        if (failed) break;
        continue;
      }
      const OpDev* op = &args.ops[slot];
      // a paired op's gather list also holds rows of its partner, tagged with their slot: those come from
      // the partner's activations (kept as the complement of the token index)
      const bool paired = op->paired != 0;
      const OpDev* pop = paired ? &args.ops[op->partner] : op;
      const unsigned char* X = static_cast<const unsigned char*>(op->x) + chunk * 16;
      const unsigned char* Xp = static_cast<const unsigned char*>(pop->x) + chunk * 16;
      const size_t pitch = (size_t)args.H * kEl;
      int tok[kPasses];
      const int n_rows = op->n_rows, n_rows_p = pop->n_rows;
      const int own_tag = paired ? slot_of(&args, slot) : 0, partner_tag = paired ? slot_of(&args, op->partner) : 0;
      bool bad = false;
#pragma unroll
      for (int j = 0; j < kPasses; ++j) {
        const int r = rbase + kRowsPerPass * j;
        const int v = r < rows ? op->gather_list[row0 + r] : 0;
        const int tag = v >> kRowSlotShift, flat = v & kRowFlatMask;
        const bool theirs = tag != own_tag;
        // an index the plan never wrote is reported below and its row is skipped
        const bool in_range = v >= 0 && (tag == own_tag || tag == partner_tag) && flat < (theirs ? n_rows_p : n_rows);
        bad |= r < rows && !in_range;
        tok[j] = (r < rows && in_range) ? (theirs ? ~(flat / args.k) : flat / args.k) : INT_MIN;
      }
      if (bad) report(c.st, MOE_EBOUNDS, slot_of(&args, slot), row0, rows, 0);
      bool fail = false;
      for (int kb = 0; kb < kblocks; ++kb, ++kiter) {
        const int stage = (int)(kiter % kNS);
        if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->empty[stage], ((kiter / kNS) & 1u) ^ 1u, 14))) { fail = true; break; }
        const unsigned sA = smem_u32(stages + (size_t)stage * kSB);
        const unsigned char* Xk = X + (size_t)kb * kRowBytes;
        const unsigned char* Xpk = Xp + (size_t)kb * kRowBytes;
#pragma unroll
        for (int j = 0; j < kPasses; ++j) {
          const int r = rbase + kRowsPerPass * j;
          // the swizzle XORs the 16-byte chunk index with the row's position in its 8-row group
          const int sw = kRowBytes == 128 ? (r & 7) : ((r >> 1) & 3);
          const int t = tok[j];
          if (t != INT_MIN)
            cp_async_16(sA + r * kRowBytes + ((chunk ^ sw) << 4),
                        (t >= 0 ? Xk : Xpk) + (size_t)(t >= 0 ? t : ~t) * pitch);
        }
        cp_async_arrive_noinc(&sc->fullA[stage]);
      }
      if (fail) break;
    }
    cp_async_wait_all();
  } else if (warp == 2) {
    MOE_REGS_DEC();
    // ============================================================ committer
    // Publishes a tile once all epilogue threads have arrived on the tile's barrier: the
    // barrier orders their stores before this warp's fence and release (cumulativity).
    int islot = 0;
    unsigned iph = 0;
    while (true) {
      if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->ifull[islot], iph, 16))) break;
      TileInfo ti;
      if (lane == 0) ti = sc->info[islot];
      const int kind = __shfl_sync(0xffffffffu, lane == 0 ? ti.kind : 0, 0);
      if (kind == kEnd) break;
      if (!__all_sync(0xffffffffu, mbar_wait(c, &sc->done[islot], iph, 17))) break;
      if (lane == 0) {
        commit_tile(c, rh, ti);
        mbar_arrive(&sc->iempty[islot]);
      }
      __syncwarp();
      if (++islot == kRing) { islot = 0; iph ^= 1u; }
    }
  } else if (warp >= 8) {
    MOE_REGS_INC();
    // ============================================================ epilogue (8 warps)
    // Warp w may read TMEM lanes 32 (w % 4) .. +31, i.e. accumulator rows of that quadrant.
    // The two warps of a quadrant split the columns of every accumulator the tile used.
    const int q = warp & 3;
    const int half = (warp - 8) >> 2;             // which half of the columns
    const int etid = threadIdx.x - 256;           // 0..255
    int islot = 0;
    unsigned iph = 0, aph[2] = {0, 0}, eph = 0, xph = 0;
    AccUse accs;
    unsigned char* scratch = sc->epi_scratch[warp - 8];
    const int srow = lane >> 2, schunk = lane & 3;          // this lane's part of a store
    while (true) {
      if (!__all_sync(0xffffffffu, mbar_wait_inline(c, &sc->ifull[islot], iph, 9))) break;
      const TileInfo ti = sc->info[islot];
      if (ti.kind == kEnd) break;
      OpDev* op = &args.ops[ti.slot];
      bool ok = true;
      if (ti.kind == kCombine) {
        combine_tokens(op, ti.row0, ti.row0 + ti.rows, args.k, args.H, etid, 256);
      } else if (kFp8) {
        ok = epilogue_fp8(c, sc, op, ti, tmem, warp, lane, eph, xph);
      } else {
        bool use[2];
        accs.take(ti.rows, use[0], use[1]);
        const bool pair = use[0] && use[1];
        const bool g1 = ti.kind != kDown;
        const int passes = (g1 ? kTileN1 : kTileN2) / 64;      // 32-column passes per warp
        const size_t pitch = (size_t)(g1 ? args.I : args.H) * 2;
#pragma unroll
        for (int b = 0; b < 2; ++b) {
          if (!use[b]) continue;
          ok = __all_sync(0xffffffffu, mbar_wait_inline(c, &sc->tfull[b], aph[b], 10));
          if (!ok) break;
          aph[b] ^= 1u;
          tc_fence_after();
          const int rbase = pair ? b * kTileM : 0;               // first tile row of this accumulator
          const int nrows = min(ti.rows - rbase, kTileM);
          if (q * 32 < nrows) {
            // 32 output columns (64 bytes of bf16) per pass.  Each lane owns one accumulator
            // row; the warp transposes the pass through its shared-memory scratch so that a
            // store instruction writes 8 rows x 64 contiguous bytes instead of 32 x 16.
            const unsigned taddr = tmem + (unsigned)b * kAccCols + ((unsigned)(q * 32) << 16);
            unsigned char* out = reinterpret_cast<unsigned char*>(g1 ? (void*)op->A : (void*)op->D) +
                                 (size_t)(ti.row0 + rbase + q * 32) * pitch +
                                 (size_t)ti.n * (g1 ? kTileN1 : kTileN2) * 2;
            const int rows_here = min(32, nrows - q * 32);
            // The TMEM load of pass p+1 is issued as soon as pass p has been converted, so its
            // latency hides behind the transpose and the stores of pass p.
            unsigned g[32], u[32];
            tc_ld32(taddr + (half * passes) * 32 + (g1 ? 0 : 0), g);
            if (g1) tc_ld32(taddr + 128 + (half * passes) * 32, u);
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
                if (g1) tc_ld32(taddr + 128 + (pass + 1) * 32, u);
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
          mbar_arrive(&sc->tempty[b]);            // accumulator may be overwritten
        }
      }
      if (!ok) break;
      mbar_arrive(&sc->done[islot]);              // this thread's part of the tile is stored
      if (++islot == kRing) { islot = 0; iph ^= 1u; }
    }
  }

  else {
    MOE_REGS_DEC();        // warp 3: idle, but its warpgroup changes its allowance together
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
  cudaError_t e = cudaFuncSetAttribute(moe_apk_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)kSmemBytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(moe_apk_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)kSmemBytes);
}

cudaError_t launch_run(const RunArgs& args, RunHead* rh, int n_ctas, cudaStream_t stream) {
  if (args.dtype == MOE_DTYPE_FP8_E4M3) moe_apk_kernel<true><<<n_ctas, kThreads, kSmemBytes, stream>>>(args, rh);
  else moe_apk_kernel<false><<<n_ctas, kThreads, kSmemBytes, stream>>>(args, rh);
  return cudaGetLastError();
}

}  // namespace moe
