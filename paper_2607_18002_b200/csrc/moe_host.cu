// Host side of the C ABI: argument validation, the layout of the caller's workspace,
// TMA descriptors, and the launches.  No hidden host synchronisation except where the
// header says so.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "moe_dev.cuh"

namespace moe {
cudaError_t launch_plan(const OpDev* d_op, Global* g, int slot, int T, int k, int E, int NT1,
                        int NT2, int work_rows, cudaStream_t stream);
cudaError_t launch_plan_masked(const OpDev* d_op, Global* g, int slot, int E, int NT1, int NT2, int slab_rows, int work_rows,
                               cudaStream_t stream);
cudaError_t launch_plan_pair(const OpDev* dp, const OpDev* pp, const OpDev* d, const OpDev* p, int* gather_m, int* comb_d,
                             int* comb_p, int Rd, int Rp, int E, int NT1, int NT2, int work_rows, int carrier_rows,
                             int slot_d, int slot_p, cudaStream_t stream);
cudaError_t launch_combine(const OpDev* d_op, int T, int k, int H, cudaStream_t stream);
cudaError_t prepare_run_kernel();
cudaError_t launch_run(const RunArgs& args, RunHead* rh, int n_ctas, cudaStream_t stream);
cudaError_t prepare_pair_kernel();
cudaError_t prepare_plan_kernels();
cudaError_t launch_pair(const RunArgs& args, RunHead* rh, int n_ctas, cudaStream_t stream);
}  // namespace moe

using namespace moe;

namespace {

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Layout {
  size_t global_off, ops_off, runzero_off, runzero_bytes, log_off, slots_off, slot_stride;
  // inside a slot
  size_t A_off, D_off, mtiles_off, tiles_off, hist_off, plan_off;
  size_t ptiles_off, pgather_off, pcomb_off, pplan_off;   // paired form: queue list, shared-space permutation, plan state
  // inside the run-zero region (after RunHead)
  size_t rs_stride;      // RunState + g1_done[max_mtiles], per slot
  size_t total;
  int max_rows, max_mtiles, max_tiles, NT1, NT2;
};

int check_config(const moe_config_t* c) {
  if (!c) return MOE_EINVAL;
  if (c->n_experts < 1 || c->n_experts > kMaxExperts) return MOE_EINVAL;
  if (c->top_k < 1 || c->top_k > 32 || c->top_k > c->n_experts) return MOE_EINVAL;
  if (c->hidden < kTileN2 || c->hidden % kTileN2) return MOE_EINVAL;
  if (c->inter < kTileN1 || c->inter % kTileN1) return MOE_EINVAL;
  // a queue entry keeps its n-tile index in eight bits
  if (c->inter / kTileN1 > 255 || c->hidden / kTileN2 > 255) return MOE_EINVAL;
  if (c->dtype != MOE_DTYPE_BF16 && c->dtype != MOE_DTYPE_FP8_E4M3) return MOE_EINVAL;
  if (c->max_tokens_per_op < 1 || c->max_ops < 1 || c->max_ops > kMaxOps) return MOE_EINVAL;
  // a flat routed index must fit below bit kRowSlotShift (the paired form tags it with a slot above that)
  if ((long long)c->max_tokens_per_op * c->top_k >= (1ll << kRowSlotShift)) return MOE_EINVAL;
  // the combine addresses the rows of the down-GEMM output by 32-bit offsets in 16-byte units
  if ((long long)c->max_tokens_per_op * c->top_k * (c->hidden / 8) >= (1ll << 32)) return MOE_EINVAL;
  if (c->wait_limit_us < 0 || c->tile_log_entries < 0 || c->n_ctas < 0) return MOE_EINVAL;
  return MOE_OK;
}

Layout make_layout(const moe_config_t* c) {
  Layout L{};
  const size_t E = c->n_experts, H = c->hidden, I = c->inter;
  L.max_rows = c->max_tokens_per_op * c->top_k;
  L.max_mtiles = (L.max_rows + kTileM - 1) / kTileM + c->n_experts;
  L.NT1 = (int)(I / kTileN1);
  L.NT2 = (int)(H / kTileN2);
  // combine entries of the largest op: small batches use smaller combine tiles
  const int small_t = c->max_tokens_per_op < kCombineSmallBatch ? c->max_tokens_per_op : kCombineSmallBatch;
  const int comb_small = (small_t + kCombineTokensSmall - 1) / kCombineTokensSmall;
  const int comb_large = (c->max_tokens_per_op + kCombineTokens - 1) / kCombineTokens;
  const int max_comb = comb_small > comb_large ? comb_small : comb_large;
  L.max_tiles = L.max_mtiles * (L.NT1 + L.NT2) + max_comb;
  const size_t n_chunks = ((size_t)L.max_rows + kPlanChunk - 1) / kPlanChunk;

  size_t off = 0;
  L.A_off = off;       off = align_up(off + (size_t)L.max_rows * I * 2, 1024);
  L.D_off = off;       off = align_up(off + (size_t)L.max_rows * H * 2, 1024);
  L.mtiles_off = off;  off = align_up(off + (size_t)L.max_mtiles * sizeof(MTile), 1024);
  L.tiles_off = off;   off = align_up(off + (size_t)L.max_tiles * sizeof(int4), 1024);
  L.hist_off = off;    off = align_up(off + 2 * n_chunks * E * 4, 1024);   // histogram + base ranks
  L.plan_off = off;    off = align_up(off + sizeof(PlanState), 1024);
  L.ptiles_off = off;  off = align_up(off + (size_t)L.max_tiles * sizeof(int4), 1024);
  L.pgather_off = off; off = align_up(off + (size_t)L.max_rows * 4, 1024);
  L.pcomb_off = off;   off = align_up(off + (size_t)L.max_rows * 4, 1024);
  L.pplan_off = off;   off = align_up(off + sizeof(PlanState), 1024);
  L.slot_stride = off;

  size_t g = 0;
  L.global_off = g;    g = align_up(g + sizeof(Global), 1024);
  L.ops_off = g;       g = align_up(g + sizeof(OpDev) * 2 * c->max_ops, 1024);   // plain and paired descriptors
  L.runzero_off = g;
  L.rs_stride = align_up(sizeof(RunState) + (size_t)L.max_mtiles * 4, 16);
  L.runzero_bytes = align_up(sizeof(RunHead) + L.rs_stride * c->max_ops, 1024);
  g += L.runzero_bytes;
  L.log_off = g;       g = align_up(g + (size_t)c->tile_log_entries * sizeof(moe_tile_rec_t), 1024);
  L.slots_off = g;
  L.total = g + L.slot_stride * c->max_ops;
  return L;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

struct moe_ctx {
  moe_config_t cfg;
  Layout L;
  unsigned char* ws;
  int n_ctas, sm_count;
  bool pair_kernel;             // bf16 on an even grid: tiles run on CTA pairs (cta_group::2)
  bool poison;                  // debug: the scratch of every op of a launch is filled with NaN patterns first
  EncodeTiledFn encode;
  moe_op_t ops[kMaxOps];
  bool planned[kMaxOps];
  OpDev host_ops[kMaxOps];      // what the device copy of each slot holds (tensor maps included)
  bool uploaded[kMaxOps];
  OpDev host_pair[kMaxOps];     // what the device copy of each slot's paired descriptor holds
  bool pair_uploaded[kMaxOps];
  int pair_of[kMaxOps];         // slot paired with this one by moe_plan_pair since both were last planned, or -1
  bool ran_paired[kMaxOps];     // the slot's last moe_run used its paired form (moe_combine follows it)
  Global* g() const { return reinterpret_cast<Global*>(ws + L.global_off); }
  RunHead* rh() const { return reinterpret_cast<RunHead*>(ws + L.runzero_off); }
  unsigned char* slot_base(int s) const { return ws + L.slots_off + L.slot_stride * s; }
  OpDev* op_dev(int s) const { return reinterpret_cast<OpDev*>(ws + L.ops_off) + s; }
  unsigned char* rs_base(int s) const { return ws + L.runzero_off + sizeof(RunHead) + L.rs_stride * s; }
};

namespace {

// 2-D tensor map (bf16, or e4m3 bytes): `rows` x `cols` row-major, box = box_rows x kBlockK columns, swizzle
// as wide as a box row
int make_map(moe_ctx* ctx, CUtensorMap* out, const void* base, size_t rows, size_t cols,
             int box_rows) {
  const bool fp8 = ctx->cfg.dtype == MOE_DTYPE_FP8_E4M3;
  const size_t el = fp8 ? 1 : 2;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * el};
  cuuint32_t box[2] = {(cuuint32_t)(kRowBytes / el), (cuuint32_t)box_rows};   // 128 bytes per box row
  cuuint32_t estr[2] = {1, 1};
  CUresult r = ctx->encode(out, fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                           const_cast<void*>(base), dims,
                           strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           kRowBytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? MOE_OK : MOE_ECUDA;
}

// a stream-ordered 4-byte write: the value travels in the launch, not through host memory
__global__ void set_word_kernel(int* p, int v) { *reinterpret_cast<volatile int*>(p) = v; }

// The op descriptor travels as a kernel parameter (no pageable-memory copy on the stream).
__global__ void write_op_kernel(const __grid_constant__ OpDev src, OpDev* dst) {
  const int n = (int)(sizeof(OpDev) / sizeof(int));
  const int* s = reinterpret_cast<const int*>(&src);
  int* d = reinterpret_cast<int*>(dst);
  for (int i = threadIdx.x; i < n; i += blockDim.x) d[i] = s[i];
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace

extern "C" {

const char* moe_strerror(int code) {
  switch (code) {
    case MOE_OK: return "ok";
    case MOE_EINVAL: return "invalid argument";
    case MOE_ENOSPC: return "workspace or slot capacity too small";
    case MOE_ECUDA: return "CUDA call failed (is there a device?)";
    case MOE_ETIMEOUT: return "a device-side wait ran out";
    case MOE_EBADID: return "expert id out of range";
    case MOE_EBOUNDS: return "device-side index check failed";
    case MOE_ENOTPLANNED: return "slot has no plan";
    default: return "unknown error";
  }
}

int moe_workspace_bytes(const moe_config_t* cfg, size_t* out) {
  if (!out) return MOE_EINVAL;
  const int rc = check_config(cfg);
  if (rc) return rc;
  *out = make_layout(cfg).total;
  return MOE_OK;
}

int moe_create(const moe_config_t* cfg, void* dev_workspace, size_t bytes, moe_ctx_t** out) {
  if (!out || !dev_workspace) return MOE_EINVAL;
  int rc = check_config(cfg);
  if (rc) return rc;
  if (reinterpret_cast<uintptr_t>(dev_workspace) & 1023) return MOE_EINVAL;
  Layout L = make_layout(cfg);
  if (bytes < L.total) return MOE_ENOSPC;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOE_ECUDA;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return MOE_ECUDA;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn)
    return MOE_ECUDA;
  if (prepare_run_kernel() != cudaSuccess || prepare_pair_kernel() != cudaSuccess ||
      prepare_plan_kernels() != cudaSuccess)
    return MOE_ECUDA;
  moe_ctx* ctx = new (std::nothrow) moe_ctx();
  if (!ctx) return MOE_ENOSPC;
  ctx->cfg = *cfg;
  if (ctx->cfg.wait_limit_us == 0) ctx->cfg.wait_limit_us = 2000000;
  ctx->L = L;
  ctx->ws = static_cast<unsigned char*>(dev_workspace);
  ctx->sm_count = sms;
  ctx->n_ctas = cfg->n_ctas > 0 ? cfg->n_ctas : sms;
  // MOE_APK_SINGLE_CTA=1 in the environment keeps bf16 on the one-CTA-per-tile kernel (for comparisons)
  const char* single = getenv("MOE_APK_SINGLE_CTA");
  ctx->pair_kernel = cfg->dtype == MOE_DTYPE_BF16 && ctx->n_ctas >= 2 && ctx->n_ctas % 2 == 0 &&
                     !(single && single[0] == '1');
  // MOE_APK_POISON=1: a row of the intermediate or of the expert output that a launch fails to write then shows
  // as NaN in y instead of passing for whatever the previous launch left there
  const char* poison = getenv("MOE_APK_POISON");
  ctx->poison = poison && poison[0] == '1';
  ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
  memset(ctx->planned, 0, sizeof(ctx->planned));
  memset(ctx->uploaded, 0, sizeof(ctx->uploaded));
  memset(ctx->ran_paired, 0, sizeof(ctx->ran_paired));
  memset(ctx->pair_uploaded, 0, sizeof(ctx->pair_uploaded));
  for (int s = 0; s < kMaxOps; ++s) ctx->pair_of[s] = -1;
  // zero the control blocks (status, budget, run state, plan states)
  cudaError_t e = cudaMemset(ctx->ws, 0, L.slots_off);
  for (int s = 0; s < cfg->max_ops && e == cudaSuccess; ++s) {
    e = cudaMemset(ctx->slot_base(s) + L.plan_off, 0, sizeof(PlanState));
    if (e == cudaSuccess) e = cudaMemset(ctx->slot_base(s) + L.pplan_off, 0, sizeof(PlanState));
  }
  if (e != cudaSuccess) { delete ctx; return MOE_ECUDA; }
  *out = ctx;
  return MOE_OK;
}

void moe_destroy(moe_ctx_t* ctx) { delete ctx; }

int moe_sm_count(moe_ctx_t* ctx) { return ctx ? ctx->sm_count : MOE_EINVAL; }
int moe_ctas_per_tile(moe_ctx_t* ctx) { return ctx ? (ctx->pair_kernel ? 2 : 1) : MOE_EINVAL; }

int moe_plan(moe_ctx_t* ctx, int slot, const moe_op_t* op, void* stream) {
  if (!ctx || !op) return MOE_EINVAL;
  const moe_config_t& c = ctx->cfg;
  if (slot < 0 || slot >= c.max_ops) return MOE_EINVAL;
  if (op->cls != MOE_CLASS_DECODE && op->cls != MOE_CLASS_PREFILL) return MOE_EINVAL;
  const bool masked = op->layout == MOE_LAYOUT_MASKED;
  if (op->layout != MOE_LAYOUT_GATHERED && !masked) return MOE_EINVAL;
  if (op->n_tokens < 0) return MOE_EINVAL;
  if (!masked && op->n_tokens > c.max_tokens_per_op) return MOE_ENOSPC;
  if (op->after_op < -1 || op->after_op >= c.max_ops || op->after_op == slot) return MOE_EINVAL;
  if (op->notify && op->notify_after < 1) return MOE_EINVAL;
  if (op->decode_sms < 0) return MOE_EINVAL;
  if (!op->counts || !op->offsets) return MOE_EINVAL;
  if (!op->w_gate_up || !op->w_down || !aligned16(op->w_gate_up) || !aligned16(op->w_down)) return MOE_EINVAL;
  if (c.dtype == MOE_DTYPE_FP8_E4M3 && (!op->s_gate_up || !op->s_down || ((op->n_tokens > 0 || masked) && !op->x_scale)))
    return MOE_EINVAL;
  if (masked) {
    if (op->slab_rows < 1 || !op->x || !op->y || !aligned16(op->x) || !aligned16(op->y)) return MOE_EINVAL;
    // the slabs of the intermediate live in the slot's scratch, one row per slab row
    if ((long long)c.n_experts * op->slab_rows > (long long)c.max_tokens_per_op * c.top_k) return MOE_ENOSPC;
  } else if (op->n_tokens > 0) {
    if (!op->x || !op->topk_ids || !op->topk_w || !op->y || !op->sorted_to_flat || !op->flat_to_sorted)
      return MOE_EINVAL;
    if (!aligned16(op->x) || !aligned16(op->y)) return MOE_EINVAL;
  }
  const Layout& L = ctx->L;
  unsigned char* sb = ctx->slot_base(slot);
  OpDev h;
  memset(&h, 0, sizeof(h));
  h.cls = op->cls;
  h.n_tokens = masked ? 0 : op->n_tokens;                     // a masked op has no token-order output to combine
  h.n_rows = masked ? c.n_experts * op->slab_rows : op->n_tokens * c.top_k;
  h.after_op = op->after_op;
  h.x = op->x; h.x_scale = op->x_scale; h.topk_ids = op->topk_ids; h.topk_w = op->topk_w;
  h.w_gate_up = op->w_gate_up; h.w_down = op->w_down; h.s_gate_up = op->s_gate_up; h.s_down = op->s_down;
  h.y = op->y; h.counts = op->counts; h.offsets = op->offsets;
  h.sorted_to_flat = op->sorted_to_flat; h.flat_to_sorted = op->flat_to_sorted;
  h.ready = op->ready; h.done = op->done;
  h.notify = op->notify; h.notify_after = op->notify_after;
  h.op_budget = op->decode_sms;
  h.A = reinterpret_cast<__nv_bfloat16*>(sb + L.A_off);
  h.a_scale = reinterpret_cast<float*>(sb + L.A_off + align_up((size_t)L.max_rows * c.inter, 16));
  // masked layout: the expert outputs ARE the op's output, in the slab layout of x
  h.D = masked ? static_cast<__nv_bfloat16*>(op->y) : reinterpret_cast<__nv_bfloat16*>(sb + L.D_off);
  h.masked = masked ? 1 : 0;
  h.mtiles = reinterpret_cast<MTile*>(sb + L.mtiles_off);
  h.tile_list = reinterpret_cast<int4*>(sb + L.tiles_off);
  h.plan_hist = reinterpret_cast<int*>(sb + L.hist_off);
  h.plan_base = h.plan_hist + (((size_t)L.max_rows + kPlanChunk - 1) / kPlanChunk) * c.n_experts;
  h.plan = reinterpret_cast<PlanState*>(sb + L.plan_off);
  h.run = reinterpret_cast<RunState*>(ctx->rs_base(slot));
  h.g1_done = reinterpret_cast<int*>(ctx->rs_base(slot) + sizeof(RunState));
  h.status = &ctx->g()->status;
  h.gather_list = op->sorted_to_flat;
  h.comb_index = op->flat_to_sorted;
  h.space_rows = h.n_rows;
  h.paired = 0;
  h.partner = -1;
  // a new plan for the slot ends any pairing it was part of
  if (ctx->pair_of[slot] >= 0) ctx->pair_of[ctx->pair_of[slot]] = -1;
  ctx->pair_of[slot] = -1;
  ctx->ran_paired[slot] = false;
  // Re-planning a slot with the same buffers (the usual serving loop) reuses the descriptors
  // already on the device: encoding seven tensor maps and uploading them is host time.
  const bool same = ctx->uploaded[slot] && memcmp(&ctx->ops[slot], op, sizeof(moe_op_t)) == 0;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!same) {
    int rc = MOE_OK;
    if (op->n_tokens > 0 || masked) {
      rc = make_map(ctx, &h.tm_a8, h.A, (size_t)L.max_rows, (size_t)c.inter, 8);
      if (!rc) rc = make_map(ctx, &h.tm_a32, h.A, (size_t)L.max_rows, (size_t)c.inter, 32);
      if (!rc) rc = make_map(ctx, &h.tm_a128, h.A, (size_t)L.max_rows, (size_t)c.inter, 128);
      if (!rc) rc = make_map(ctx, &h.tm_a256, h.A, (size_t)L.max_rows, (size_t)c.inter, 256);
      if (!rc) rc = make_map(ctx, &h.tm_w1, op->w_gate_up, (size_t)c.n_experts * 2 * c.inter, (size_t)c.hidden, 128);
      if (!rc) rc = make_map(ctx, &h.tm_w1h, op->w_gate_up, (size_t)c.n_experts * 2 * c.inter, (size_t)c.hidden, 64);
      if (!rc) rc = make_map(ctx, &h.tm_w2, op->w_down, (size_t)c.n_experts * c.hidden, (size_t)c.inter, 128);
      if (masked) {
        const size_t xr = (size_t)c.n_experts * op->slab_rows;
        if (!rc) rc = make_map(ctx, &h.tm_x8, op->x, xr, (size_t)c.hidden, 8);
        if (!rc) rc = make_map(ctx, &h.tm_x32, op->x, xr, (size_t)c.hidden, 32);
        if (!rc) rc = make_map(ctx, &h.tm_x128, op->x, xr, (size_t)c.hidden, 128);
        if (!rc) rc = make_map(ctx, &h.tm_x256, op->x, xr, (size_t)c.hidden, 256);
      }
      if (rc) return rc;
    }
    ctx->planned[slot] = false;
    write_op_kernel<<<1, 128, 0, st>>>(h, ctx->op_dev(slot));
    if (cudaGetLastError() != cudaSuccess) { ctx->uploaded[slot] = false; return MOE_ECUDA; }
    ctx->host_ops[slot] = h;
    ctx->ops[slot] = *op;             // what the device copy of the slot now describes
    ctx->uploaded[slot] = true;
  }
  const int work_rows = c.dtype == MOE_DTYPE_FP8_E4M3 ? kWorkRowsFp8 : kWorkRowsBf16;
  const cudaError_t pe = masked ? launch_plan_masked(ctx->op_dev(slot), ctx->g(), slot, c.n_experts, L.NT1, L.NT2,
                                                     op->slab_rows, work_rows, st)
                                : launch_plan(ctx->op_dev(slot), ctx->g(), slot, op->n_tokens, c.top_k, c.n_experts, L.NT1,
                                              L.NT2, work_rows, st);
  if (pe != cudaSuccess) {
    ctx->planned[slot] = false;
    return MOE_ECUDA;
  }
  ctx->planned[slot] = true;
  return MOE_OK;
}

int moe_run(moe_ctx_t* ctx, const int32_t* slots, int n_ops, int fuse_combine, void* stream) {
  if (!ctx || !slots || n_ops < 1 || n_ops > ctx->cfg.max_ops) return MOE_EINVAL;
  const moe_config_t& c = ctx->cfg;
  RunArgs a;
  memset(&a, 0, sizeof(a));
  for (int i = 0; i < n_ops; ++i) {
    const int s = slots[i];
    if (s < 0 || s >= c.max_ops) return MOE_EINVAL;
    if (!ctx->planned[s]) return MOE_ENOTPLANNED;
    for (int j = 0; j < i; ++j) if (slots[j] == s) return MOE_EINVAL;
    a.slots[i] = s;
  }
  // a slot whose pair partner is in the same launch runs in its paired form
  a.n_slots = c.max_ops;
  for (int s = 0; s < kMaxOps; ++s) a.desc[s] = (signed char)s;
  for (int i = 0; i < n_ops; ++i) {
    const int s = slots[i], q = ctx->pair_of[s];
    bool both = false;
    for (int j = 0; j < n_ops && q >= 0; ++j) both |= slots[j] == q;
    ctx->ran_paired[s] = both;
    if (both) {
      a.slots[i] = c.max_ops + s;
      a.desc[s] = (signed char)(c.max_ops + s);
    }
  }
  for (int i = 0; i < n_ops; ++i) {      // after_op must name an op of this run
    const int dep = ctx->ops[slots[i]].after_op;
    if (dep < 0) continue;
    bool found = false;
    for (int j = 0; j < n_ops; ++j) found |= slots[j] == dep;
    if (!found) return MOE_EINVAL;
  }
  a.g = ctx->g();
  a.ops = ctx->op_dev(0);
  a.log = reinterpret_cast<moe_tile_rec_t*>(ctx->ws + ctx->L.log_off);
  a.log_cap = c.tile_log_entries;
  a.n_ops = n_ops;
  a.fuse_combine = fuse_combine ? 1 : 0;
  a.E = c.n_experts; a.k = c.top_k; a.H = c.hidden; a.I = c.inter;
  a.dtype = c.dtype;
  a.kb_elems = c.dtype == MOE_DTYPE_FP8_E4M3 ? 128 : kBlockK;
  a.wait_ns = (long long)c.wait_limit_us * 1000;
  a.static_kind = -1;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(ctx->rh(), 0, ctx->L.runzero_bytes, st) != cudaSuccess) return MOE_ECUDA;
  if (ctx->poison) {
    for (int i = 0; i < n_ops; ++i) {
      unsigned char* sb = ctx->slot_base(slots[i]);
      const size_t a_bytes = ctx->L.D_off - ctx->L.A_off, d_bytes = ctx->L.mtiles_off - ctx->L.D_off;
      if (cudaMemsetAsync(sb + ctx->L.A_off, 0xff, a_bytes, st) != cudaSuccess) return MOE_ECUDA;
      if (cudaMemsetAsync(sb + ctx->L.D_off, 0xff, d_bytes, st) != cudaSuccess) return MOE_ECUDA;
    }
  }
  const cudaError_t le = ctx->pair_kernel ? launch_pair(a, ctx->rh(), ctx->n_ctas, st)
                                          : launch_run(a, ctx->rh(), ctx->n_ctas, st);
  if (le != cudaSuccess) return MOE_ECUDA;
  return MOE_OK;
}

int moe_run_plain(moe_ctx_t* ctx, int slot, void* stream) {
  if (!ctx || slot < 0 || slot >= ctx->cfg.max_ops) return MOE_EINVAL;
  if (!ctx->pair_kernel) return MOE_EINVAL;
  if (!ctx->planned[slot]) return MOE_ENOTPLANNED;
  if (ctx->ops[slot].after_op >= 0 || ctx->ops[slot].ready) return MOE_EINVAL;
  const moe_config_t& c = ctx->cfg;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the grid is the op's entry count, which only the device knows: wait for the plan and read it
  PlanState ps;
  if (cudaStreamSynchronize(st) != cudaSuccess) return MOE_ECUDA;
  if (cudaMemcpy(&ps, ctx->slot_base(slot) + ctx->L.plan_off, sizeof(ps), cudaMemcpyDeviceToHost) != cudaSuccess)
    return MOE_ECUDA;
  if (!ps.planned) return MOE_ENOTPLANNED;
  RunArgs a;
  memset(&a, 0, sizeof(a));
  a.slots[0] = slot;
  a.g = ctx->g();
  a.ops = ctx->op_dev(0);
  a.log = reinterpret_cast<moe_tile_rec_t*>(ctx->ws + ctx->L.log_off);
  a.log_cap = c.tile_log_entries;
  a.n_ops = 1;
  a.fuse_combine = 0;
  a.E = c.n_experts; a.k = c.top_k; a.H = c.hidden; a.I = c.inter;
  a.dtype = c.dtype;
  a.kb_elems = kBlockK;
  a.wait_ns = (long long)c.wait_limit_us * 1000;
  a.n_slots = c.max_ops;
  for (int s = 0; s < kMaxOps; ++s) a.desc[s] = (signed char)s;
  ctx->ran_paired[slot] = false;
  if (cudaMemsetAsync(ctx->rh(), 0, ctx->L.runzero_bytes, st) != cudaSuccess) return MOE_ECUDA;
  a.static_kind = 0;
  if (ps.n_gemm_tiles > 0 && launch_pair(a, ctx->rh(), 2 * ps.n_gemm_tiles, st) != cudaSuccess) return MOE_ECUDA;
  if (ctx->ops[slot].layout == MOE_LAYOUT_GATHERED &&
      launch_combine(ctx->op_dev(slot), ctx->ops[slot].n_tokens, c.top_k, c.hidden, st) != cudaSuccess)
    return MOE_ECUDA;
  return MOE_OK;
}

int moe_combine(moe_ctx_t* ctx, int slot, void* stream) {
  if (!ctx || slot < 0 || slot >= ctx->cfg.max_ops) return MOE_EINVAL;
  if (!ctx->planned[slot]) return MOE_ENOTPLANNED;
  if (ctx->ops[slot].layout != MOE_LAYOUT_GATHERED) return MOE_EINVAL;     // a masked op has nothing to combine
  // after a launch that ran the slot in its paired form, the expert outputs lie in the pair's shared row space
  const int desc = ctx->ran_paired[slot] ? ctx->cfg.max_ops + slot : slot;
  if (launch_combine(ctx->op_dev(desc), ctx->ops[slot].n_tokens, ctx->cfg.top_k, ctx->cfg.hidden,
                     static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return MOE_ECUDA;
  return MOE_OK;
}

int moe_plan_pair(moe_ctx_t* ctx, int slot_prefill, int slot_decode, int carrier_rows, void* stream) {
  if (!ctx) return MOE_EINVAL;
  const moe_config_t& c = ctx->cfg;
  const int sp = slot_prefill, sd = slot_decode;
  if (sp < 0 || sp >= c.max_ops || sd < 0 || sd >= c.max_ops || sp == sd) return MOE_EINVAL;
  if (!ctx->planned[sp] || !ctx->planned[sd]) return MOE_ENOTPLANNED;
  const moe_op_t &op = ctx->ops[sp], &od = ctx->ops[sd];
  if (op.cls != MOE_CLASS_PREFILL || od.cls != MOE_CLASS_DECODE) return MOE_EINVAL;
  if (op.layout != MOE_LAYOUT_GATHERED || od.layout != MOE_LAYOUT_GATHERED) return MOE_EINVAL;
  // one weight tile can only serve rows of both ops if both ops read the same weights
  if (op.w_gate_up != od.w_gate_up || op.w_down != od.w_down || op.s_gate_up != od.s_gate_up || op.s_down != od.s_down)
    return MOE_EINVAL;
  const bool fp8 = c.dtype == MOE_DTYPE_FP8_E4M3;
  if (carrier_rows == 0) carrier_rows = fp8 ? kWorkRowsFp8 : kWorkRowsBf16;
  if (carrier_rows != 128 && carrier_rows != 256) return MOE_EINVAL;
  const Layout& L = ctx->L;
  const long long Rp = (long long)op.n_tokens * c.top_k, Rd = (long long)od.n_tokens * c.top_k;
  if (Rp + Rd > L.max_rows) return MOE_ENOSPC;      // the shared row space lives in one slot's scratch
  if (op.n_tokens == 0 || od.n_tokens == 0) return MOE_EINVAL;
  unsigned char *bp = ctx->slot_base(sp), *bd = ctx->slot_base(sd);
  int* gather_m = reinterpret_cast<int*>(bp + L.pgather_off);
  OpDev hp = ctx->host_ops[sp], hd = ctx->host_ops[sd];
  // both paired descriptors address the prefill slot's scratch (A, its scales, D) as the shared row space
  hd.A = hp.A; hd.a_scale = hp.a_scale; hd.D = hp.D;
  hd.tm_a8 = hp.tm_a8; hd.tm_a32 = hp.tm_a32; hd.tm_a128 = hp.tm_a128; hd.tm_a256 = hp.tm_a256;
  OpDev* both[2] = {&hp, &hd};
  for (int i = 0; i < 2; ++i) {
    OpDev* h = both[i];
    unsigned char* b = i == 0 ? bp : bd;
    h->tile_list = reinterpret_cast<int4*>(b + L.ptiles_off);
    h->plan = reinterpret_cast<PlanState*>(b + L.pplan_off);
    h->gather_list = gather_m;
    h->comb_index = reinterpret_cast<int*>(b + L.pcomb_off);
    h->space_rows = (int)(Rp + Rd);
    h->paired = 1;
    h->partner = c.max_ops + (i == 0 ? sd : sp);
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the usual loop pairs the same two ops on the same buffers again and again: upload only what changed
  const int which[2] = {sp, sd};
  for (int i = 0; i < 2; ++i) {
    const int s = which[i];
    if (ctx->pair_uploaded[s] && memcmp(&ctx->host_pair[s], both[i], sizeof(OpDev)) == 0) continue;
    write_op_kernel<<<1, 128, 0, st>>>(*both[i], ctx->op_dev(c.max_ops + s));
    if (cudaGetLastError() != cudaSuccess) { ctx->pair_uploaded[s] = false; return MOE_ECUDA; }
    ctx->host_pair[s] = *both[i];
    ctx->pair_uploaded[s] = true;
  }
  if (launch_plan_pair(ctx->op_dev(c.max_ops + sd), ctx->op_dev(c.max_ops + sp), ctx->op_dev(sd), ctx->op_dev(sp), gather_m,
                       reinterpret_cast<int*>(bd + L.pcomb_off), reinterpret_cast<int*>(bp + L.pcomb_off), (int)Rd, (int)Rp,
                       c.n_experts, L.NT1, L.NT2, fp8 ? kWorkRowsFp8 : kWorkRowsBf16, carrier_rows, sd, sp, st) != cudaSuccess)
    return MOE_ECUDA;
  if (ctx->pair_of[sp] >= 0) ctx->pair_of[ctx->pair_of[sp]] = -1;
  if (ctx->pair_of[sd] >= 0) ctx->pair_of[ctx->pair_of[sd]] = -1;
  ctx->pair_of[sp] = sd;
  ctx->pair_of[sd] = sp;
  return MOE_OK;
}

int moe_set_budget(moe_ctx_t* ctx, int decode_sms, void* stream) {
  if (!ctx || decode_sms < 0) return MOE_EINVAL;
  set_word_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(&ctx->g()->budget, decode_sms);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ECUDA;
}

namespace {
// q' = min(q_max, ceil_c(q * x_moe / x_star)) from the slot's planned footprint (Section 6.4)
__global__ void scaled_budget_kernel(int* budget, const PlanState* plan, int q, double x_star, int q_max, int c) {
  const double want = ceil((double)q * (double)plan->n_mtiles / x_star);
  long long v = want > 2147483000.0 ? 2147483000ll : (long long)want;
  v = (v + c - 1) / c * c;
  *budget = (int)(v < (long long)q_max ? v : (long long)q_max);
}
}  // namespace

int moe_set_budget_scaled(moe_ctx_t* ctx, int slot, int q, double x_moe_star, int q_max, void* stream) {
  if (!ctx || slot < 0 || slot >= ctx->cfg.max_ops || q < 0 || q_max < 0 || !(x_moe_star > 0.0)) return MOE_EINVAL;
  if (!ctx->planned[slot]) return MOE_ENOTPLANNED;
  const PlanState* ps = reinterpret_cast<const PlanState*>(ctx->slot_base(slot) + ctx->L.plan_off);
  scaled_budget_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(&ctx->g()->budget, ps, q, x_moe_star, q_max,
                                                                      ctx->pair_kernel ? 2 : 1);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ECUDA;
}

int moe_get_budget(moe_ctx_t* ctx, int32_t* out) {
  if (!ctx || !out) return MOE_EINVAL;
  return cudaMemcpy(out, &ctx->g()->budget, sizeof(int32_t), cudaMemcpyDeviceToHost) == cudaSuccess ? MOE_OK : MOE_ECUDA;
}

int moe_status(moe_ctx_t* ctx, int32_t* code, int32_t detail[4]) {
  if (!ctx || !code) return MOE_EINVAL;
  Status s;
  if (cudaMemcpy(&s, &ctx->g()->status, sizeof(s), cudaMemcpyDeviceToHost) != cudaSuccess) return MOE_ECUDA;
  *code = s.code;
  if (detail) for (int i = 0; i < 4; ++i) detail[i] = s.detail[i];
  // a plan that met an expert id out of range left its slot without a usable permutation
  if (s.code == MOE_EBADID && s.detail[0] >= 0 && s.detail[0] < ctx->cfg.max_ops) {
    const int bad = s.detail[0];
    ctx->planned[bad] = false;
    if (ctx->pair_of[bad] >= 0) ctx->pair_of[ctx->pair_of[bad]] = -1;
    ctx->pair_of[bad] = -1;
  }
  if (s.code != 0 || s.abort != 0)
    if (cudaMemset(&ctx->g()->status, 0, sizeof(Status)) != cudaSuccess) return MOE_ECUDA;
  return MOE_OK;
}

int moe_footprint(moe_ctx_t* ctx, int slot, int32_t* x_moe, int32_t* n_tiles) {
  if (!ctx || slot < 0 || slot >= ctx->cfg.max_ops) return MOE_EINVAL;
  if (!ctx->planned[slot]) return MOE_ENOTPLANNED;
  PlanState ps;
  if (cudaMemcpy(&ps, ctx->slot_base(slot) + ctx->L.plan_off, sizeof(ps), cudaMemcpyDeviceToHost) != cudaSuccess)
    return MOE_ECUDA;
  if (x_moe) *x_moe = ps.n_mtiles;
  if (n_tiles) *n_tiles = ps.n_gemm_tiles + ps.n_comb_tiles;
  return MOE_OK;
}

int moe_read_tile_table(moe_ctx_t* ctx, int slot, int32_t* host_out, int max_tiles) {
  if (!ctx || !host_out || slot < 0 || slot >= ctx->cfg.max_ops || max_tiles < 0) return MOE_EINVAL;
  if (!ctx->planned[slot]) return MOE_ENOTPLANNED;
  int n = max_tiles < ctx->L.max_mtiles ? max_tiles : ctx->L.max_mtiles;
  if (n > 0 && cudaMemcpy(host_out, ctx->slot_base(slot) + ctx->L.mtiles_off, (size_t)n * sizeof(MTile),
                          cudaMemcpyDeviceToHost) != cudaSuccess)
    return MOE_ECUDA;
  return MOE_OK;
}

int moe_read_tile_log(moe_ctx_t* ctx, moe_tile_rec_t* host_out, int max_records, int* n) {
  if (!ctx || !host_out || !n || max_records < 0) return MOE_EINVAL;
  RunHead rh;
  if (cudaMemcpy(&rh, ctx->rh(), sizeof(rh), cudaMemcpyDeviceToHost) != cudaSuccess) return MOE_ECUDA;
  int cnt = (int)rh.log_count;
  if (cnt > ctx->cfg.tile_log_entries) cnt = ctx->cfg.tile_log_entries;
  if (cnt > max_records) cnt = max_records;
  if (cnt > 0 && cudaMemcpy(host_out, ctx->ws + ctx->L.log_off, (size_t)cnt * sizeof(moe_tile_rec_t),
                            cudaMemcpyDeviceToHost) != cudaSuccess)
    return MOE_ECUDA;
  *n = cnt;
  return MOE_OK;
}

}  // extern "C"
