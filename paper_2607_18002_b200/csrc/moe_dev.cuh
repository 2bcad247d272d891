// Device-side data structures shared by the plan, run and combine kernels and the host
// code that lays them out inside the caller's workspace.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/moe_apk.h"

namespace moe {

constexpr int kTileM = MOE_TILE_M;   // token rows per tile (M_t)
constexpr int kTileN1 = 128;         // SwiGLU output columns per gate/up tile (256 weight rows)
constexpr int kTileN2 = 256;         // output columns per down-GEMM tile
constexpr int kBlockK = 64;          // K elements per pipeline stage (one 128-byte swizzle row of bf16)
constexpr int kRowBytes = kBlockK * 2;
constexpr int kStages = 3;           // shared-memory pipeline depth (64 KB per stage)
constexpr int kCombineTokens = 16;   // tokens per combine tile ...
constexpr int kCombineTokensSmall = 4;     // ... of an op with at most kCombineSmallBatch tokens (a decode batch): its
constexpr int kCombineSmallBatch = 1024;   // combine is a latency chain per token, so it is spread over more units
constexpr int kPlanChunk = 256;      // routed rows ranked by one warp in the plan kernels
constexpr int kGroupWork = 16;       // work tiles per dependency group of the tile list
constexpr int kWorkRowsBf16 = 256;   // rows of a work tile: two m-tiles share each weight tile
constexpr int kWorkRowsFp8 = 128;    // fp8: the accumulator and both partial buffers fill TMEM
constexpr int kMaxOps = 16;
constexpr int kMaxExperts = 1024;

// kGateUpDirect: a gate/up tile whose activation rows are consecutive rows of x (masked layout): they are
// loaded by TMA like the rows of a down tile instead of being gathered through a permutation
__host__ __device__ inline int combine_tile_tokens(int T) { return T <= kCombineSmallBatch ? kCombineTokensSmall : kCombineTokens; }

enum TileKind : int { kGateUp = 0, kDown = 1, kCombine = 2, kGateUpDirect = 3 };

// Queue entry (16 bytes, one load per claim): x = kind | n-tile << 4 | m-tile << 12,
// y = first packed row (first token for a combine tile), z = valid rows, w = expert.
__host__ __device__ inline int4 make_entry(int kind, int n, int m, int row0, int rows, int expert) {
  return make_int4(kind | (n << 4) | (m << 12), row0, rows, expert);
}
__host__ __device__ inline int entry_kind(const int4& e) { return e.x & 15; }
__host__ __device__ inline int entry_n(const int4& e) { return (e.x >> 4) & 0xff; }
__host__ __device__ inline int entry_m(const int4& e) { return (e.x >> 12) & 0xfffff; }

struct MTile {   // one row block of one expert (the unit counted by x_moe)
  int expert, row0, rows, pad;
};

// Written by the plan kernel, read by the run kernel.
struct PlanState {
  int n_mtiles;       // x_moe
  int n_gemm_tiles;   // queue entries of kind gate/up or down
  int n_comb_tiles;   // queue entries of kind combine (follow the GEMM entries)
  int planned;        // 1 after a moe_plan that accepted every expert id, else 0
  int n_extra_gemm;   // paired prefill op: GEMM entries of the decode op's list that carry rows of this op
  int pad[3];
};

// Zeroed by moe_run before every launch.
struct RunState {
  int gemm_done;      // committed GEMM tiles
  int tiles_done;     // committed tiles of any kind
  int done;           // 1 when the op has fully finished
  int pad;
};

struct Status;

struct __align__(128) OpDev {
  CUtensorMap tm_a8;    // [Rmax, I]   box {64, 8}   packed intermediate, 8 consecutive rows
  CUtensorMap tm_a32;   // [Rmax, I]   box {64, 32}
  CUtensorMap tm_w1;    // [E*2I, H]   box {64, 128} gate/up weights
  CUtensorMap tm_w2;    // [E*H, I]    box {64, 128} down weights
  CUtensorMap tm_a128;  // [Rmax, I]   box {64, 128}
  CUtensorMap tm_a256;  // [Rmax, I]   box {64, 256}
  CUtensorMap tm_w1h;   // [E*2I, H]   box {64, 64}  gate/up weights, half-height box (CTA-pair kernel)
  CUtensorMap tm_x8;    // masked layout only: x as [E*slab_rows, H], boxes of 8 / 32 / 128 / 256 rows
  CUtensorMap tm_x32;
  CUtensorMap tm_x128;
  CUtensorMap tm_x256;
  int cls, n_tokens, n_rows, after_op;
  const void* x;
  const float* x_scale;
  const int* topk_ids;
  const float* topk_w;
  const void* w_gate_up;
  const void* w_down;
  const float* s_gate_up;
  const float* s_down;
  void* y;
  int* counts;
  int* offsets;
  int* sorted_to_flat;
  int* flat_to_sorted;
  const unsigned* ready;
  unsigned* done;
  unsigned* notify;      // set once notify_after tiles of the op have committed
  int notify_after;
  int op_budget;         // > 0: written to the budget word when the op's first tile is claimed
  // workspace-owned
  __nv_bfloat16* A;      // [Rmax, I]  SwiGLU output, packed order (e4m3 bytes in the fp8 path)
  float* a_scale;        // [Rmax, I/128] fp32 scales of A (fp8 path)
  __nv_bfloat16* D;      // [Rmax, H]  expert output, packed order
  MTile* mtiles;         // [max_mtiles]
  int4* tile_list;       // [max_tiles] queue entries in claim order
  int* plan_hist;        // [n_chunks, E] per-warp histogram
  int* plan_base;        // [n_chunks, E] per-warp base rank of each expert
  PlanState* plan;
  RunState* run;
  int* g1_done;          // [max_mtiles] committed gate/up tiles per work tile
  Status* status;        // the context's device status block
  // Which list of routed rows the run kernels walk.  A plain op: its own permutation (the plan's public
  // outputs).  The paired form of a decode + prefill op that share their weights (moe_plan_pair): one row
  // space for both, every entry of the gather list tagged with the slot whose row it is.
  const int* gather_list;   // packed row -> flat routed index (paired: | slot << kRowSlotShift)
  const int* comb_index;    // flat routed index -> packed row of D
  int space_rows;           // rows of the packed space that A, D and comb_index refer to
  int masked;               // 1: masked layout (x, A, y in per-expert slabs of slab_rows rows)
  int paired;               // 1: this is the paired form of the slot
  int partner;              // paired: descriptor index of the other op of the pair, else -1
  int pad_[2];
};
constexpr int kRowSlotShift = 27;                       // a flat routed index stays below 2^27 (moe_create checks)
constexpr int kRowFlatMask = (1 << kRowSlotShift) - 1;

struct Status {   // first error wins (atomicCAS on code)
  int code;
  int detail[4];
  int abort;      // set with code; every CTA stops claiming when it sees it
  int pad[2];
};

struct Global {
  Status status;
  int budget;             // decode SM budget q (Section 6.4)
  int pad[7];
};

// Start of the region moe_run zeroes before every launch; the per-slot RunState blocks and
// g1_done arrays follow it.
struct RunHead {
  unsigned heads[2];      // next ticket of the decode / prefill queue
  unsigned log_count;
  int pad[5];
};

struct RunArgs {
  Global* g;
  OpDev* ops;             // indexed by slot
  moe_tile_rec_t* log;
  int log_cap;
  int n_ops;
  int fuse_combine;
  int E, k, H, I;
  int dtype, kb_elems;    // MOE_DTYPE_*; K elements per pipeline stage (64 bf16 / 128 e4m3)
  long long wait_ns;
  int n_slots;            // slots of the context; descriptor d >= n_slots is the paired form of slot d - n_slots
  signed char desc[kMaxOps];   // slot -> the descriptor that stands for it in this launch
  int static_kind;        // -1: persistent launch served from the queues.  >= 0: a plain launch, claiming unit u
                          // of the grid runs queue entry u of slots[0] and ends
  int slots[kMaxOps];     // descriptor indices of the launch's ops, in the order given
};

__device__ __forceinline__ int slot_of(const RunArgs* a, int desc) { return desc >= a->n_slots ? desc - a->n_slots : desc; }

__device__ __noinline__ inline void report(Status* st, int code, int d0, int d1, int d2, int d3) {
  if (atomicCAS(&st->code, 0, code) == 0) {
    st->detail[0] = d0; st->detail[1] = d1; st->detail[2] = d2; st->detail[3] = d3;
  }
  __threadfence();
  atomicExch(&st->abort, 1);
}

__device__ inline unsigned long long gtime_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

}  // namespace moe
