/*
 * moe_apk.h -- C ABI of the B200 (sm_100a) routed-MoE expert library.
 *
 * One "operation" is the routed-expert computation of one token batch of one class
 * (decode or prefill) for one MoE layer:
 *
 *     y[t,:] = sum_j w[t,j] * FFN_{ids[t,j]}(x[t,:]),
 *     FFN_e(x) = (silu(x W_gate[e]) * (x W_up[e])) W_down[e]
 *
 * (the paper's Section 2.1 MoE module; the kernel that runs it is the adaptive
 * persistent kernel of Section 4: two grouped GEMMs, the activation, the MoE pre- and
 * post-processing and the tile scheduler in one launch, Section 7.1).
 *
 * Conventions
 *   - Every pointer in moe_op_t and the workspace is a DEVICE pointer owned by the
 *     caller; the library never frees it and keeps no reference after moe_destroy.
 *     moe_config_t / moe_op_t themselves, and all `out` arguments, are HOST memory.
 *   - `stream` is a cudaStream_t passed as void*.  Calls only enqueue work; none of
 *     them synchronises the host except moe_status and moe_read_tile_log.
 *   - Row-major everywhere.  bf16 = 2-byte bfloat16, e4m3 = 1-byte OCP E4M3FN.
 *   - Return value: 0 on success, a negative MOE_E* code otherwise.  Errors that only
 *     the device can see (an expert id out of range, a wait that ran out) are recorded
 *     in a device status word and read back with moe_status after a stream sync; a
 *     kernel that hits one stops claiming tiles and returns -- it never traps or hangs.
 *   - There is no CPU fallback: without a CUDA device every compute entry point fails
 *     with MOE_ECUDA.
 *   - Debug aid: with MOE_APK_POISON=1 in the environment at moe_create, every moe_run first
 *     fills the scratch (intermediate and expert-output rows) of its ops with NaN patterns, so
 *     that a row a launch failed to write shows as NaN in y.  Off by default (it costs two
 *     large memsets per op and launch).
 */
#ifndef MOE_APK_H_
#define MOE_APK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  MOE_OK = 0,
  MOE_EINVAL = -1,   /* bad argument: NULL, shape, alignment, slot out of range          */
  MOE_ENOSPC = -2,   /* workspace too small / op larger than max_tokens_per_op           */
  MOE_ECUDA = -3,    /* a CUDA runtime or driver call failed (no device, launch error)   */
  MOE_ETIMEOUT = -4, /* device: a wait (ready word, dependency, pipeline) ran out        */
  MOE_EBADID = -5,   /* device: an expert id outside [0, n_experts)                      */
  MOE_EBOUNDS = -6,  /* device: an index check failed inside a kernel                    */
  MOE_ENOTPLANNED = -7 /* moe_run / moe_combine on a slot with no moe_plan               */
};

enum { MOE_DTYPE_BF16 = 0, MOE_DTYPE_FP8_E4M3 = 1 };
enum { MOE_CLASS_DECODE = 0, MOE_CLASS_PREFILL = 1 };
/* How an op's activations are laid out (Section 2.4).  GATHERED: x is [T, H] in token order and the
 * plan packs the routed rows per expert (the contiguous layout).  MASKED: x already sits in per-expert
 * slabs [E, slab_rows, H] of which the first counts[e] rows of slab e are valid (what a dispatch step
 * of fixed-size buffers delivers, and what decode under captured graphs uses): nothing is permuted,
 * y is written in the same slab layout and there is no combine. */
enum { MOE_LAYOUT_GATHERED = 0, MOE_LAYOUT_MASKED = 1 };

/* Height of a token-dimension tile (the M_t of the footprint formula, Section 6.2). */
#define MOE_TILE_M 128

typedef struct moe_ctx moe_ctx_t; /* opaque, host side */

typedef struct {
  int32_t n_experts;         /* E, 1..1024                                               */
  int32_t top_k;             /* k, 1..32                                                 */
  int32_t hidden;            /* H, multiple of 256                                       */
  int32_t inter;             /* I, multiple of 128                                       */
  int32_t dtype;             /* MOE_DTYPE_*                                              */
  int32_t max_tokens_per_op; /* sizes the per-slot scratch; buffers are fixed up front,  */
  int32_t max_ops;           /* as the paper's preallocated final buffers (Section 5.2); */
                             /* max_tokens_per_op * k * H must stay below 2^35           */
  int32_t wait_limit_us;     /* device-side wait budget before MOE_ETIMEOUT; 0 = 2 s     */
  int32_t tile_log_entries;  /* capacity of the per-tile log; 0 = logging off            */
  int32_t n_ctas;            /* persistent grid size; 0 = one CTA per SM                 */
} moe_config_t;

typedef struct {
  int32_t cls;      /* MOE_CLASS_DECODE (priority) or MOE_CLASS_PREFILL                   */
  int32_t n_tokens; /* T >= 0                                                             */
  const void* x;          /* [T, H] bf16 | e4m3                                           */
  const float* x_scale;   /* [T, H/128] fp32 (e4m3 only, else NULL)                       */
  const int32_t* topk_ids;/* [T, k] expert ids                                            */
  const float* topk_w;    /* [T, k] router weights                                        */
  const void* w_gate_up;  /* [E, 2I, H]: rows 0..I-1 gate, I..2I-1 up; K (=H) contiguous  */
  const void* w_down;     /* [E, H, I]; K (=I) contiguous                                 */
  const float* s_gate_up; /* [E, 2I/128, H/128] fp32 block scales (e4m3 only, else NULL)  */
  const float* s_down;    /* [E, H/128, I/128]                                            */
  void* y;                /* [T, H] bf16 output                                           */
  int32_t* counts;        /* [E]    out: rows per expert                                  */
  int32_t* offsets;       /* [E+1]  out: exclusive prefix sum, offsets[E] = T*k           */
  int32_t* sorted_to_flat;/* [T*k]  out: packed row p -> flat routed index i = t*k + j    */
  int32_t* flat_to_sorted;/* [T*k]  out: inverse permutation                              */
  const uint32_t* ready;  /* optional: the op may be scheduled once *ready != 0           */
  uint32_t* done;         /* optional: set to 1 when the op's last tile has committed     */
  int32_t after_op;       /* -1, or a slot (of the same moe_run) that must finish first   */
  int32_t notify_after;   /* with `notify`: 1 .. the op's tile count                      */
  uint32_t* notify;       /* optional: set to 1 (system scope) once notify_after tiles of */
                          /* this op have committed -- e.g. the ready word of another op, */
                          /* which then arrives while this one is being served            */
  int32_t decode_sms;     /* the SM budget field of the op template (Section 4.2): > 0    */
                          /* makes the decode budget take this value when the op's first  */
                          /* tile is claimed, 0 leaves the budget word alone              */
  int32_t layout;         /* MOE_LAYOUT_*.  MASKED: n_tokens is ignored; x and y are       */
  int32_t slab_rows;      /* [E, slab_rows, H] (x_scale [E, slab_rows, H/128]); counts [E] */
                          /* is an INPUT (valid rows per slab, 0..slab_rows); offsets is   */
                          /* still written; topk_ids, topk_w and the permutations are not  */
                          /* used; E * slab_rows <= max_tokens_per_op * top_k              */
} moe_op_t;

/* One record per executed tile (only when tile_log_entries > 0). Times are GPU
 * globaltimer nanoseconds; the preemption-interval analysis of Section 7.6 is made
 * from these. */
typedef struct {
  uint64_t t_claim;  /* the tile was taken from its queue                                 */
  uint64_t t_commit; /* its outputs are written and published                             */
  int32_t slot;      /* op slot                                                           */
  int32_t tile;      /* index in the op's tile list                                       */
  int16_t cls, kind; /* class; 0 = gate/up GEMM + SwiGLU, 1 = down GEMM, 2 = combine,     */
                     /* 3 = gate/up GEMM + SwiGLU of a masked-layout op                   */
  int16_t cta, sm;   /* CTA index and SM id that ran it (first CTA of a pair)                */
} moe_tile_rec_t;

/* Bytes of device workspace moe_create needs for this configuration. */
int moe_workspace_bytes(const moe_config_t* cfg, size_t* out);

/* Builds a context on the current device.  dev_workspace: device memory, 1024-byte
 * aligned, at least moe_workspace_bytes(); the library zeroes what it needs (on the
 * legacy default stream, synchronously). */
int moe_create(const moe_config_t* cfg, void* dev_workspace, size_t bytes, moe_ctx_t** out);
void moe_destroy(moe_ctx_t* ctx);

/* Plan (pre-processing): top-k ids -> counts, exclusive offsets by a device prefix
 * sum, the stable permutation (rows of an expert keep ascending flat index -- the
 * packed per-expert layout of Section 2.4), and the op's tile table, whose length is
 * the footprint x_moe = sum_{e: m_e>0} ceil(m_e / M_t) of Section 6.2.  Binds `op` to
 * `slot`; the struct is copied, the buffers it names must stay valid until the work
 * enqueued on them has finished.
 * An expert id outside [0, n_experts) is recorded as MOE_EBADID (detail: slot, flat
 * index, id).  Such a row gets no packed position: flat_to_sorted[i] = -1, the unclaimed
 * tail of sorted_to_flat is -1, counts and offsets cover the accepted rows only, and the
 * slot is left without a plan -- moe_run and moe_combine enqueued behind it do nothing for
 * it, and once moe_status has returned the error they answer MOE_ENOTPLANNED until the
 * slot is planned again. */
int moe_plan(moe_ctx_t* ctx, int slot, const moe_op_t* op, void* stream);

/* The persistent expert kernel over the planned ops in `slots` (one launch): every CTA
 * repeatedly claims the next tile from the decode queue or the prefill queue of
 * Section 4.2 -- CTAs with index below the decode budget prefer decode tiles, the
 * others prefill tiles, each falling back to the other class when its own has nothing
 * ready (Section 6.4) -- and runs it: gate/up grouped GEMM with fused SwiGLU, then the
 * down grouped GEMM, on rows gathered through the permutation.  A phase switch happens
 * only between tiles (Section 4.2), so results do not depend on the schedule.
 * Ops of one class are served in the order given.  With fuse_combine != 0 the
 * router-weighted combine runs as tiles of the same launch and y is final when the
 * kernel ends; otherwise call moe_combine.
 * An op without tokens has no tiles: it counts as finished as soon as the op it comes
 * after has (at once if there is none), its done and notify words are set then, and its
 * ready word is not consulted.
 * `ready`, `done` and `notify` words may also live in pinned host memory that the device
 * can address (they are read and written at system scope), so the host can make an op
 * ready, or learn of progress, while the kernel runs; every device-side wait on them is
 * bounded by wait_limit_us. */
int moe_run(moe_ctx_t* ctx, const int32_t* slots, int n_ops, int fuse_combine, void* stream);

/* Pairs a prefill op and a decode op that share their expert weights (both planned, same w_gate_up /
 * w_down / scale pointers) so that a launch running both streams an expert's weight tile ONCE for rows of
 * both: the decode op's rows of an expert travel in "carrier" tiles together with the ragged tail of that
 * expert's prefill rows (what its full prefill tiles leave over) when the tail fits into the decode rows'
 * last tile of `carrier_rows` rows (128 or 256; 0 = the kernel's work-tile height: 256 for bf16, 128 for e4m3,
 * where a 256-row carrier runs as two 128-row tiles that follow one another).  Carrier tiles belong to the decode class -- decode priority and the budget work as before
 * (Sections 4.2, 6.4) -- and the prefill op keeps the remaining rows.  A row's arithmetic does not depend
 * on the tile it sits in, so y of both ops is bit-identical to the unpaired launch; counts, offsets and the
 * permutations of moe_plan are untouched (the shared row space is private workspace).
 *   - call after moe_plan of both slots, on the same stream; a later moe_plan of either slot ends the pairing;
 *   - moe_run uses the paired form when BOTH slots are in the launch, the plain form otherwise;
 *   - the prefill op is complete (done word, successors, its combine tiles) only when the decode op's GEMM
 *     tiles are, because some of them carry its rows: a decode op that never becomes ready holds it back;
 *   - n_tokens of both ops together must fit max_tokens_per_op (the shared row space lives in one slot's
 *     scratch), else MOE_ENOSPC; both ops need at least one token (MOE_EINVAL). */
int moe_plan_pair(moe_ctx_t* ctx, int slot_prefill, int slot_decode, int carrier_rows, void* stream);

/* The same tiles as a plain (non-persistent) launch, for measuring what the tile scheduler costs
 * (the scheduling-overhead experiment of Section 7.4): ONE launch with one claiming unit per queue
 * entry of the op in `slot` -- unit u runs entry u and ends; no queue, no budget, no ready word; a
 * down tile waits, bounded, for the gate/up tiles of its rows, which belong to units with a lower
 * index -- then the stand-alone combine.  Same tile code, bit-identical y.  bf16 on an even grid only
 * (MOE_EINVAL otherwise, and for an op with a ready word or a predecessor).  The grid size is the
 * op's entry count, which lives on the device: this call SYNCHRONISES the stream to read it, so it
 * is a measuring tool, not a serving path. */
int moe_run_plain(moe_ctx_t* ctx, int slot, void* stream);

/* Post-processing: y[t,:] = sum_j w[t,j] * D[flat_to_sorted[t*k+j],:], slots added in
 * order j = 0..k-1 in fp32 (the last step of the MoE module of Section 2.1).  A permutation
 * entry outside [0, T*k) is reported as MOE_EBOUNDS and contributes nothing. */
int moe_combine(moe_ctx_t* ctx, int slot, void* stream);

/* Decode SM budget q of Section 6.4: a stream-ordered 4-byte write to the device word
 * the running kernel reads at every tile boundary.  0 <= decode_sms. */
int moe_set_budget(moe_ctx_t* ctx, int decode_sms, void* stream);

/* Online SM reallocation (Section 6.4, "Online SM Reallocation"): sets the budget word to
 *     q' = min(q_max, ceil_c(q * x_moe / x_moe_star))
 * where x_moe is the footprint of the decode op planned in `slot` (read on the device: the call
 * is stream-ordered after that moe_plan and never synchronises), x_moe_star > 0 the footprint the
 * static budget q was chosen for, and ceil_c rounds up to a multiple of c = moe_ctas_per_tile
 * (the claiming unit: the paper's CTA cluster).  The product and quotient are taken in double
 * precision.  MOE_ENOTPLANNED if the slot has no plan, MOE_EINVAL for q < 0, q_max < 0 or
 * x_moe_star <= 0. */
int moe_set_budget_scaled(moe_ctx_t* ctx, int slot, int q, double x_moe_star, int q_max, void* stream);

/* Reads the budget word back (synchronous copy; call after synchronising the stream). */
int moe_get_budget(moe_ctx_t* ctx, int32_t* out);

/* Device status (synchronous copy; call after synchronising the stream).  code is 0 or
 * a MOE_E* value; detail[0..3] describe where (meaning depends on code).  Clears it. */
int moe_status(moe_ctx_t* ctx, int32_t* code, int32_t detail[4]);

/* Footprint of a planned slot: x_moe (tiles of height MOE_TILE_M) and the number of
 * queue entries.  Synchronous copy; call after synchronising the stream. */
int moe_footprint(moe_ctx_t* ctx, int slot, int32_t* x_moe, int32_t* n_tiles);

/* Copies the slot's tile table (x_moe entries of {expert, first packed row, rows, 0})
 * to host memory.  Synchronous. */
int moe_read_tile_table(moe_ctx_t* ctx, int slot, int32_t* host_out, int max_tiles);

/* Copies up to max_records tile records of the last moe_run to host memory and
 * returns how many were written in *n.  Synchronous. */
int moe_read_tile_log(moe_ctx_t* ctx, moe_tile_rec_t* host_out, int max_records, int* n);

/* The plan step for callers that must not allocate (no counterpart in the paper: it is a
 * deployment convenience of this library).  Same counts / offsets / sorted_to_flat /
 * flat_to_sorted as moe_plan, bit for bit, but without a context or a workspace: the
 * histogram scratch is a fixed 128 KB device array inside the library image, held by every
 * GPU that loads the library until the process exits.  It is meant for code that runs where
 * a device allocation is not an option -- all memory belongs to another allocator, or the
 * caller may not make calls that can synchronise the device, as cudaMalloc and cudaFree
 * can.  The call itself allocates nothing and calls no allocating routine.
 *   - limits: n_tokens * top_k <= MOE_PLAN_STATIC_MAX_ROWS and n_experts <=
 *     MOE_PLAN_STATIC_MAX_EXPERTS, else MOE_ENOSPC (nothing is launched);
 *   - all pointers are device pointers owned by the caller, sizes as in moe_op_t;
 *   - `stream` must belong to the device that is current when the call is made: the
 *     scratch array's address is looked up on the current device;
 *   - expert ids outside [0, n_experts) are skipped silently (moe_plan reports them);
 *   - every call looks up the scratch array's device address (nothing is cached, so a device
 *     reset between calls is harmless); the first look-up on a device may load the library's
 *     device code: make that first call outside any stream capture;
 *   - every call uses the same array, which keeps the previous call's contents (nothing
 *     in it needs clearing between calls); calls whose kernels could overlap on the GPU
 *     -- other streams, other host threads -- race on it and must be serialised. */
#define MOE_PLAN_STATIC_MAX_ROWS 32768
#define MOE_PLAN_STATIC_MAX_EXPERTS 256
int moe_plan_static(const int32_t* topk_ids, int32_t n_tokens, int32_t top_k, int32_t n_experts,
                    int32_t* counts, int32_t* offsets, int32_t* sorted_to_flat,
                    int32_t* flat_to_sorted, void* stream);

/* The router ahead of moe_plan (Section 2.1: a router selects the top-k routed experts of each
 * token; the arithmetic is this library's reading -- softmax over the experts, the k largest,
 * weights renormalised over those k).  logits [T, E] fp32 -> topk_ids [T, k] (in order of
 * decreasing logit, ties to the lower expert id) and topk_w [T, k] fp32 (they sum to 1).  All
 * pointers are device pointers; no context, no workspace.  n_experts <= 1024, top_k <= 32 and
 * <= n_experts, else MOE_EINVAL.  Logits must be finite. */
int moe_route(const float* logits, int32_t n_tokens, int32_t n_experts, int32_t top_k,
              int32_t* topk_ids, float* topk_w, void* stream);

/* Multiprocessor count of the context's device (the default persistent grid). */
int moe_sm_count(moe_ctx_t* ctx);

/* How many CTAs work on one tile: 2 when the context runs bf16 on an even grid (tiles are
 * then claimed and run by pairs of CTAs on neighbouring SMs, one tcgen05 MMA spanning both),
 * else 1.  The claiming unit of Section 4.2 is that group: the decode budget of
 * moe_set_budget still counts CTAs (a pair is inside the budget when its first CTA is), and
 * tile records carry the CTA index and SM id of the group's first CTA.  Setting
 * MOE_APK_SINGLE_CTA=1 in the environment before moe_create keeps every context at 1. */
int moe_ctas_per_tile(moe_ctx_t* ctx);

const char* moe_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* MOE_APK_H_ */
