// Scheduling pieces shared by the persistent kernels: bounded waits, the two-class tile queue
// (Sections 4.2 and 6.4), tile publication and the SwiGLU helper.
#pragma once
#include "moe_dev.cuh"
#include "moe_ptx.cuh"

namespace moe {

constexpr int kRing = 4;                               // tile-info ring depth
constexpr int kEnd = -1;
constexpr int kClaimAt = 2;                             // claim the next tile after this k-block
constexpr int kPublishLead = 5;                         // try to hand the next tile on from this many k-blocks before the end

struct TileInfo {
  int kind, slot, tile, m, row0, rows, n, kblocks, expert, cls;
  unsigned long long t_claim;
};

// per-class queue tables of one launch (built once per CTA in shared memory)
struct QueueTables {
  int n_cls[2];
  int cls_slot[2][kMaxOps];
  int cls_free[2][kMaxOps];        // 1: the op has no ready word and no predecessor
  unsigned cum[2][kMaxOps + 1];
};

// ------------------------------------------------------------------ bounded waits
struct Ctx {
  const RunArgs* a;
  Status* st;
};

__device__ __forceinline__ bool aborted(const Ctx& c) { return ld_volatile(&c.st->abort) != 0; }

// where: a small code telling which wait gave up (reported in detail[0])
__device__ __noinline__ inline bool mbar_wait_slow(const Ctx& c, void* bar, unsigned parity, int where) {
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

// the same wait without any function call: for code that keeps many registers live across it
__device__ __forceinline__ bool mbar_wait_inline(const Ctx& c, void* bar, unsigned parity, int where) {
  unsigned long long t0 = 0;
  for (unsigned it = 0;; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 63u) == 63u) {
      if (aborted(c)) return false;
      const unsigned long long now = gtime_ns();
      if (t0 == 0) t0 = now;
      else if ((long long)(now - t0) > c.a->wait_ns) {
        if (atomicCAS(&c.st->code, 0, MOE_ETIMEOUT) == 0) {
          c.st->detail[0] = where; c.st->detail[1] = (int)blockIdx.x;
          c.st->detail[2] = (int)threadIdx.x; c.st->detail[3] = (int)parity;
        }
        __threadfence();
        atomicExch(&c.st->abort, 1);
        return false;
      }
    }
  }
}

// spin until *p >= target (acquire); one thread
__device__ __noinline__ inline bool wait_counter(const Ctx& c, const int* p, int target, int where) {
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
// a slot whose plan was rejected (an expert id out of range) holds no tiles
__device__ __forceinline__ int op_total_tiles(const OpDev* op, int fuse) {
  if (op->plan->planned == 0) return 0;
  return op->plan->n_gemm_tiles + op->plan->n_extra_gemm + (fuse ? op->plan->n_comb_tiles : 0);
}
// entries of the op's own queue list
__device__ __forceinline__ int op_queue_entries(const OpDev* op, int fuse) {
  if (op->plan->planned == 0) return 0;
  return op->plan->n_gemm_tiles + (fuse ? op->plan->n_comb_tiles : 0);
}
// GEMM entries that must have committed before the op's combine may run
__device__ __forceinline__ int op_gemm_tiles(const OpDev* op) { return op->plan->n_gemm_tiles + op->plan->n_extra_gemm; }

// An op without tiles (no tokens, or a plan that was rejected) never commits anything: it counts as
// finished as soon as its own predecessor has, and its ready word is not consulted.
__device__ inline bool op_finished(const RunArgs* a, int slot) {
  for (int hop = 0; slot >= 0 && hop <= kMaxOps; ++hop) {
    const OpDev* op = &a->ops[a->desc[slot]];
    if (op_total_tiles(op, a->fuse_combine) > 0) return ld_acquire(&op->run->done) != 0;
    slot = op->after_op;
  }
  return true;
}

__device__ inline bool op_ready(const RunArgs* a, const OpDev* op) {
  if (op->ready != nullptr && ld_acquire_sys(op->ready) == 0) return false;
  return op_finished(a, op->after_op);
}

// Marks as done every tile-less op of the run whose chain of predecessors ends at `finished`
// (-1: at no op at all) through tile-less ops only.  One thread; called at kernel start and when an
// op's last tile commits.
__device__ inline void finish_empty_ops(const RunArgs* a, int finished) {
  for (int i = 0; i < a->n_ops; ++i) {
    OpDev* op = &a->ops[a->slots[i]];
    if (op_total_tiles(op, a->fuse_combine) > 0) continue;
    int dep = op->after_op;
    for (int hop = 0; dep >= 0 && hop <= kMaxOps && op_total_tiles(&a->ops[a->desc[dep]], a->fuse_combine) == 0; ++hop)
      dep = a->ops[dep].after_op;
    if (dep != finished) continue;
    atomicExch(&op->run->done, 1);
    if (op->done != nullptr) st_release_sys(op->done, 1u);
    if (op->notify != nullptr) st_release_sys(op->notify, 1u);
  }
}

// Claim by the whole producer warp.  1: claimed (ti filled), 0: queue exhausted, -1: the op
// at the head of the queue is not ready.  The head is only peeked before the fetch-add, so no
// CTA can be starved by others (a compare-and-swap loop starves the SMs far from the counter);
// the price is that a ticket can land just past an op boundary, in an op that is not ready
// yet -- the caller then waits for it (bounded), holding only tickets whose predecessors in
// the queue are all claimed already.
__device__ inline int try_claim(const RunArgs* a, QueueTables* sc, RunHead* rh, int cls, unsigned h,
                                int lane, TileInfo& ti, bool& need_ready) {
  const int n = sc->n_cls[cls];
  if (n == 0) return 0;
  const unsigned total = sc->cum[cls][n];
  h = __shfl_sync(0xffffffffu, h, 0);       // one peek for the whole warp: lanes index entries by it
  if (h >= total) return 0;
  int i = 0;
  while (h >= sc->cum[cls][i + 1]) ++i;
  int slot = sc->cls_slot[cls][i];
  const OpDev* op = &a->ops[slot];
  const unsigned base = h - sc->cum[cls][i];
  // Everything the warp branches on comes from ONE lane's loads: the lanes of this warp run apart after a
  // sleep, and words such as an op's done flag or the GEMM counter change between one lane's load and the next's.
  int takeable = 1;
  if (lane == 0) {
    if (!sc->cls_free[cls][i] && !op_ready(a, op)) takeable = 0;
    // The head stands at the op's combine entries while GEMM entries they depend on are still running
    // (other units hold them; for a paired prefill op, the decode list's carrier tiles): nothing to take here
    // yet -- the caller turns to the other class instead of holding a combine ticket it cannot run.
    else if (base >= (unsigned)op->plan->n_gemm_tiles && ld_acquire(&op->run->gemm_done) < op_gemm_tiles(op)) takeable = 0;
  }
  if (__shfl_sync(0xffffffffu, takeable, 0) == 0) return -1;
  // the 32 entries from the head on are fetched while the fetch-add is in flight
  const unsigned n_op = sc->cum[cls][i + 1] - sc->cum[cls][i];
  int4 e = make_int4(0, 0, 0, 0);
  if (base + lane < n_op) e = op->tile_list[base + lane];
  unsigned t = 0;
  if (lane == 0) t = atomicAdd(&rh->heads[cls], 1u);
  t = __shfl_sync(0xffffffffu, t, 0);
  if (t >= total) return 0;
  need_ready = false;
  // the prefetched entries belong to the op at the peeked head: usable only while the ticket stays in it
  const bool same_op = t < sc->cum[cls][i + 1];
  if (!same_op) {                          // past the op boundary: a later op of the class
    while (t >= sc->cum[cls][i + 1]) ++i;
    slot = sc->cls_slot[cls][i];
    op = &a->ops[slot];
    need_ready = !sc->cls_free[cls][i];
  }
  const unsigned local = t - sc->cum[cls][i];
  // the op is instantiated by the claim of its first tile: its budget field takes effect now
  if (local == 0 && lane == 0 && op->op_budget > 0) atomicExch(&a->g->budget, op->op_budget);
  const unsigned d = t - h;
  const bool hit = same_op && d < 32u;
  int4 got;
  got.x = __shfl_sync(0xffffffffu, e.x, hit ? d : 0);
  got.y = __shfl_sync(0xffffffffu, e.y, hit ? d : 0);
  got.z = __shfl_sync(0xffffffffu, e.z, hit ? d : 0);
  got.w = __shfl_sync(0xffffffffu, e.w, hit ? d : 0);
  if (!hit) got = op->tile_list[local];
  ti.kind = entry_kind(got);
  ti.n = entry_n(got);
  ti.m = entry_m(got);
  ti.row0 = got.y;
  ti.rows = got.z;
  ti.expert = got.w;
  ti.slot = slot;
  ti.tile = (int)local;
  ti.cls = cls;
  ti.kblocks = ti.kind == kCombine ? 0 : (ti.kind == kDown ? a->I : a->H) / a->kb_elems;
  return 1;
}

// One pass of the decision at a tile boundary (whole producer warp): 1 = claimed, 0 = both
// queues exhausted, -1 = something exists but is not ready yet.  The abort word, the budget
// word and both queue heads are loaded together (one round trip), then at most one
// fetch-add per class.
__device__ inline int claim_once(const Ctx& c, QueueTables* sc, RunHead* rh, int lane, TileInfo& ti,
                                 bool& need_ready) {
  const RunArgs* a = c.a;
  // one lane reads the words and the warp takes ITS values: the budget word, the abort word and the heads
  // change while the kernel runs, and the lanes do not load them at the same instant
  int ab = 0, q = 0;
  unsigned h0 = 0, h1 = 0;
  if (lane == 0) {
    ab = ld_volatile(&c.st->abort);
    q = ld_volatile(&a->g->budget);
    h0 = *reinterpret_cast<volatile unsigned*>(&rh->heads[0]);
    h1 = *reinterpret_cast<volatile unsigned*>(&rh->heads[1]);
  }
  ab = __shfl_sync(0xffffffffu, ab, 0);
  q = __shfl_sync(0xffffffffu, q, 0);
  h0 = __shfl_sync(0xffffffffu, h0, 0);
  h1 = __shfl_sync(0xffffffffu, h1, 0);
  if (ab != 0) return 0;
  const int first = ((int)blockIdx.x < q) ? MOE_CLASS_DECODE : MOE_CLASS_PREFILL;
  need_ready = false;
  const int r1 = try_claim(a, sc, rh, first, first == 0 ? h0 : h1, lane, ti, need_ready);
  int r2 = 0;
  if (r1 != 1) r2 = try_claim(a, sc, rh, 1 - first, first == 0 ? h1 : h0, lane, ti, need_ready);
  if (r1 == 1 || r2 == 1) {
    ti.t_claim = gtime_ns();
    return 1;
  }
  return (r1 == 0 && r2 == 0) ? 0 : -1;
}

// A ticket that landed in an op that is not ready yet: wait for it (bounded).  Whole warp; lane 0 looks and
// decides, so that all lanes leave together.
__device__ inline bool wait_op_ready(const Ctx& c, int lane, const TileInfo& ti) {
  const RunArgs* a = c.a;
  const unsigned long long w0 = gtime_ns();
  while (true) {
    int r = 0;                                   // 1: ready, -1: give up
    if (lane == 0) {
      if (op_ready(a, &a->ops[ti.slot])) r = 1;
      else if (aborted(c)) r = -1;
      else if ((long long)(gtime_ns() - w0) > a->wait_ns) {
        report(c.st, MOE_ETIMEOUT, 11, (int)blockIdx.x, slot_of(a, ti.slot), ti.tile);
        r = -1;
      }
    }
    r = __shfl_sync(0xffffffffu, r, 0);
    if (r != 0) return r > 0;
    __nanosleep(256);
  }
}

// The plain (non-persistent) launch: unit `unit` of the grid takes queue entry `unit` of the run's only op
// and nothing else.  No queue head, no budget, no ready word.  A down tile still waits (bounded) for the
// gate/up tiles of its rows: they sit earlier in the list, i.e. in units with a lower index.
__device__ inline void claim_static(const RunArgs* a, int unit, TileInfo& ti) {
  const int slot = a->slots[0];
  const OpDev* op = &a->ops[slot];
  ti.kind = kEnd;
  if (unit >= op->plan->n_gemm_tiles) return;
  const int4 got = op->tile_list[unit];
  ti.kind = entry_kind(got);
  ti.n = entry_n(got);
  ti.m = entry_m(got);
  ti.row0 = got.y;
  ti.rows = got.z;
  ti.expert = got.w;
  ti.slot = slot;
  ti.tile = unit;
  ti.cls = op->cls;
  ti.kblocks = (ti.kind == kDown ? a->I : a->H) / a->kb_elems;
  ti.t_claim = gtime_ns();
}

// Blocking form: waits (bounded) while an op exists that is not ready.  Returns with
// ti.kind == kEnd when nothing is left (or the run was aborted).
__device__ inline void claim_next(const Ctx& c, QueueTables* sc, RunHead* rh, int lane, TileInfo& ti,
                                  bool& need_ready) {
  unsigned long long t0 = 0;
  for (unsigned it = 0;; ++it) {
    const int r = claim_once(c, sc, rh, lane, ti, need_ready);
    if (r == 1) return;
    if (r == 0) break;
    __nanosleep(256);                         // an op exists but is not ready yet
    if ((it & 15u) == 15u) {                  // lane 0's clock decides for the warp
      int expired = 0;
      if (lane == 0) {
        const unsigned long long now = gtime_ns();
        if (t0 == 0) t0 = now;
        else if ((long long)(now - t0) > c.a->wait_ns) {
          report(c.st, MOE_ETIMEOUT, 1, (int)blockIdx.x, 0, 0);
          expired = 1;
        }
      }
      if (__shfl_sync(0xffffffffu, expired, 0)) break;
    }
  }
  ti.kind = kEnd;
}

// one committed entry counted for `op` (descriptor `desc`): counters, notify word, completion
__device__ inline void count_commit(const RunArgs* a, OpDev* op, int desc, bool gemm) {
  if (gemm) atomicAdd(&op->run->gemm_done, 1);
  const int done = atomicAdd(&op->run->tiles_done, 1) + 1;
  if (op->notify != nullptr && done == op->notify_after) st_release_sys(op->notify, 1u);
  if (done == op_total_tiles(op, a->fuse_combine)) {
    __threadfence();
    atomicExch(&op->run->done, 1);
    if (op->done != nullptr) st_release_sys(op->done, 1u);
    finish_empty_ops(a, slot_of(a, desc));
  }
}

// Publishing a finished tile: dependency counter, op completion, done word, log.
// Called by one thread after all writers of the tile have fenced and synchronised.
__device__ inline void commit_tile(const Ctx& c, RunHead* rh, const TileInfo& ti) {
  const RunArgs* a = c.a;
  OpDev* op = &a->ops[ti.slot];
  __threadfence();
  fence_async_proxy();
  const unsigned long long t_commit = a->log_cap > 0 ? gtime_ns() : 0ull;   // before it is published
  if (ti.kind == kGateUp || ti.kind == kGateUpDirect) atomicAdd(&op->g1_done[ti.m], 1);
  count_commit(a, op, ti.slot, ti.kind != kCombine);
  // a GEMM entry of a paired decode op carries rows of the prefill op too: it counts for both
  if (op->paired && op->cls == MOE_CLASS_DECODE && ti.kind != kCombine) count_commit(a, &a->ops[op->partner], op->partner, true);
  if (a->log_cap > 0) {
    const unsigned idx = atomicAdd(&rh->log_count, 1u);
    if (idx < (unsigned)a->log_cap) {
      moe_tile_rec_t r;
      r.t_claim = ti.t_claim;
      r.t_commit = t_commit;
      r.slot = slot_of(a, ti.slot);
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

__device__ inline void build_queues(const RunArgs* a, QueueTables* sc) {
  sc->n_cls[0] = sc->n_cls[1] = 0;
  sc->cum[0][0] = sc->cum[1][0] = 0;
  for (int i = 0; i < a->n_ops; ++i) {
    const int slot = a->slots[i];
    const OpDev* op = &a->ops[slot];
    const int cls = op->cls;
    const int j = sc->n_cls[cls]++;
    sc->cls_slot[cls][j] = slot;
    sc->cls_free[cls][j] = (op->ready == nullptr && op->after_op < 0) ? 1 : 0;
    sc->cum[cls][j + 1] = sc->cum[cls][j] + (unsigned)op_queue_entries(op, a->fuse_combine);
  }
}

// silu(g) * u through the hardware tanh approximation (one special-function op per element;
// its error, |g| * 2.4e-4 at worst, stays below the bf16 rounding of the result)
__device__ __forceinline__ float silu_mul(float g, float u) {
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * g));
  const float hg = 0.5f * g;
  return fmaf(hg, t, hg) * u;                     // g * sigmoid(g) = g/2 * (1 + tanh(g/2))
}

}  // namespace moe
