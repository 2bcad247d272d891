"""Python binding of the routed-MoE expert library (sm_100a, C ABI in include/moe_apk.h).

Argument marshalling only: every step of the path (plan, persistent expert kernel,
combine, budget write) runs in the CUDA library.  PyTorch appears here solely as the
owner of device memory and streams.  There is no CPU fallback: if the shared object is
missing or no CUDA device is present the calls raise.

The functions carry the C names (moe_plan, moe_run, moe_combine, moe_set_budget, ...);
`Context` and `bind_op` are thin conveniences that keep the tensors an op points to
alive and fill the C structs from them.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmoe_apk.so")

MOE_OK, MOE_EINVAL, MOE_ENOSPC, MOE_ECUDA = 0, -1, -2, -3
MOE_ETIMEOUT, MOE_EBADID, MOE_EBOUNDS, MOE_ENOTPLANNED = -4, -5, -6, -7
MOE_DTYPE_BF16, MOE_DTYPE_FP8_E4M3 = 0, 1
MOE_CLASS_DECODE, MOE_CLASS_PREFILL = 0, 1
MOE_LAYOUT_GATHERED, MOE_LAYOUT_MASKED = 0, 1
MOE_TILE_M = 128

EXPORTS = ("moe_workspace_bytes", "moe_create", "moe_destroy", "moe_plan", "moe_run",
           "moe_combine", "moe_set_budget", "moe_set_budget_scaled", "moe_get_budget", "moe_status", "moe_footprint",
           "moe_read_tile_table", "moe_read_tile_log", "moe_sm_count", "moe_ctas_per_tile", "moe_strerror",
           "moe_plan_static", "moe_route", "moe_run_plain", "moe_plan_pair")
MOE_PLAN_STATIC_MAX_ROWS, MOE_PLAN_STATIC_MAX_EXPERTS = 32768, 256


class MoeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


class moe_config_t(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "n_experts", "top_k", "hidden", "inter", "dtype", "max_tokens_per_op", "max_ops",
        "wait_limit_us", "tile_log_entries", "n_ctas")]


class moe_op_t(C.Structure):
    _fields_ = [("cls", C.c_int32), ("n_tokens", C.c_int32),
                ("x", C.c_void_p), ("x_scale", C.c_void_p),
                ("topk_ids", C.c_void_p), ("topk_w", C.c_void_p),
                ("w_gate_up", C.c_void_p), ("w_down", C.c_void_p),
                ("s_gate_up", C.c_void_p), ("s_down", C.c_void_p),
                ("y", C.c_void_p),
                ("counts", C.c_void_p), ("offsets", C.c_void_p),
                ("sorted_to_flat", C.c_void_p), ("flat_to_sorted", C.c_void_p),
                ("ready", C.c_void_p), ("done", C.c_void_p),
                ("after_op", C.c_int32), ("notify_after", C.c_int32), ("notify", C.c_void_p),
                ("decode_sms", C.c_int32), ("layout", C.c_int32), ("slab_rows", C.c_int32)]


class moe_tile_rec_t(C.Structure):
    _fields_ = [("t_claim", C.c_uint64), ("t_commit", C.c_uint64),
                ("slot", C.c_int32), ("tile", C.c_int32),
                ("cls", C.c_int16), ("kind", C.c_int16), ("cta", C.c_int16), ("sm", C.c_int16)]


TILE_REC_DTYPE = np.dtype([("t_claim", "<u8"), ("t_commit", "<u8"), ("slot", "<i4"),
                           ("tile", "<i4"), ("cls", "<i2"), ("kind", "<i2"), ("cta", "<i2"),
                           ("sm", "<i2")])

_lib = None


def lib() -> C.CDLL:
    """The loaded C-ABI library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2607_18002_b200.build` "
                "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        vp, i32 = C.c_void_p, C.c_int32
        L.moe_workspace_bytes.argtypes = [C.POINTER(moe_config_t), C.POINTER(C.c_size_t)]
        L.moe_create.argtypes = [C.POINTER(moe_config_t), vp, C.c_size_t, C.POINTER(vp)]
        L.moe_destroy.argtypes = [vp]
        L.moe_destroy.restype = None
        L.moe_plan.argtypes = [vp, C.c_int, C.POINTER(moe_op_t), vp]
        L.moe_run.argtypes = [vp, C.POINTER(i32), C.c_int, C.c_int, vp]
        L.moe_combine.argtypes = [vp, C.c_int, vp]
        L.moe_run_plain.argtypes = [vp, C.c_int, vp]
        L.moe_plan_pair.argtypes = [vp, C.c_int, C.c_int, C.c_int, vp]
        L.moe_set_budget.argtypes = [vp, C.c_int, vp]
        L.moe_set_budget_scaled.argtypes = [vp, C.c_int, C.c_int, C.c_double, C.c_int, vp]
        L.moe_get_budget.argtypes = [vp, C.POINTER(i32)]
        L.moe_status.argtypes = [vp, C.POINTER(i32), C.POINTER(i32)]
        L.moe_footprint.argtypes = [vp, C.c_int, C.POINTER(i32), C.POINTER(i32)]
        L.moe_read_tile_table.argtypes = [vp, C.c_int, vp, C.c_int]
        L.moe_read_tile_log.argtypes = [vp, vp, C.c_int, C.POINTER(C.c_int)]
        L.moe_plan_static.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp]
        L.moe_route.argtypes = [vp, i32, i32, i32, vp, vp, vp]
        L.moe_sm_count.argtypes = [vp]
        L.moe_ctas_per_tile.argtypes = [vp]
        L.moe_strerror.argtypes = [C.c_int]
        L.moe_strerror.restype = C.c_char_p
        for name in EXPORTS:
            if name not in ("moe_destroy", "moe_strerror"):
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().moe_strerror(int(code)).decode()


def _check(rc: int, where: str) -> None:
    if rc != 0:
        raise MoeError(rc, where)


# ------------------------------------------------------------------ the C entry points

def moe_workspace_bytes(cfg: moe_config_t) -> int:
    out = C.c_size_t()
    _check(lib().moe_workspace_bytes(C.byref(cfg), C.byref(out)), "moe_workspace_bytes")
    return int(out.value)


def moe_create(cfg: moe_config_t, dev_workspace_ptr: int, nbytes: int) -> int:
    ctx = C.c_void_p()
    _check(lib().moe_create(C.byref(cfg), C.c_void_p(dev_workspace_ptr), nbytes, C.byref(ctx)),
           "moe_create")
    return ctx.value


def moe_destroy(ctx: int) -> None:
    lib().moe_destroy(C.c_void_p(ctx))


def moe_plan(ctx: int, slot: int, op: moe_op_t, stream: int) -> None:
    _check(lib().moe_plan(C.c_void_p(ctx), slot, C.byref(op), C.c_void_p(stream)), "moe_plan")


def moe_run(ctx: int, slots: Sequence[int], fuse_combine: bool, stream: int) -> None:
    arr = (C.c_int32 * len(slots))(*slots)
    _check(lib().moe_run(C.c_void_p(ctx), arr, len(slots), int(bool(fuse_combine)),
                         C.c_void_p(stream)), "moe_run")


def moe_plan_pair(ctx: int, slot_prefill: int, slot_decode: int, carrier_rows: int, stream: int) -> None:
    _check(lib().moe_plan_pair(C.c_void_p(ctx), slot_prefill, slot_decode, carrier_rows, C.c_void_p(stream)),
           "moe_plan_pair")


def moe_run_plain(ctx: int, slot: int, stream: int) -> None:
    _check(lib().moe_run_plain(C.c_void_p(ctx), slot, C.c_void_p(stream)), "moe_run_plain")


def moe_combine(ctx: int, slot: int, stream: int) -> None:
    _check(lib().moe_combine(C.c_void_p(ctx), slot, C.c_void_p(stream)), "moe_combine")


def moe_set_budget(ctx: int, decode_sms: int, stream: int) -> None:
    _check(lib().moe_set_budget(C.c_void_p(ctx), int(decode_sms), C.c_void_p(stream)),
           "moe_set_budget")


def moe_set_budget_scaled(ctx: int, slot: int, q: int, x_moe_star: float, q_max: int, stream: int) -> None:
    _check(lib().moe_set_budget_scaled(C.c_void_p(ctx), int(slot), int(q), float(x_moe_star), int(q_max),
                                       C.c_void_p(stream)), "moe_set_budget_scaled")


def moe_get_budget(ctx: int) -> int:
    out = C.c_int32()
    _check(lib().moe_get_budget(C.c_void_p(ctx), C.byref(out)), "moe_get_budget")
    return int(out.value)


def moe_status(ctx: int):
    code = C.c_int32()
    detail = (C.c_int32 * 4)()
    _check(lib().moe_status(C.c_void_p(ctx), C.byref(code), detail), "moe_status")
    return int(code.value), [int(v) for v in detail]


def moe_footprint(ctx: int, slot: int):
    x, n = C.c_int32(), C.c_int32()
    _check(lib().moe_footprint(C.c_void_p(ctx), slot, C.byref(x), C.byref(n)), "moe_footprint")
    return int(x.value), int(n.value)


def moe_read_tile_table(ctx: int, slot: int) -> np.ndarray:
    x_moe, _ = moe_footprint(ctx, slot)
    out = np.zeros((max(x_moe, 1), 4), dtype=np.int32)
    _check(lib().moe_read_tile_table(C.c_void_p(ctx), slot, out.ctypes.data_as(C.c_void_p), x_moe),
           "moe_read_tile_table")
    return out[:x_moe]


def moe_read_tile_log(ctx: int, max_records: int) -> np.ndarray:
    out = np.zeros(max(max_records, 1), dtype=TILE_REC_DTYPE)
    n = C.c_int()
    _check(lib().moe_read_tile_log(C.c_void_p(ctx), out.ctypes.data_as(C.c_void_p), max_records,
                                   C.byref(n)), "moe_read_tile_log")
    return out[:n.value]


def moe_plan_static(topk_ids_ptr: int, n_tokens: int, top_k: int, n_experts: int, counts_ptr: int,
                    offsets_ptr: int, sorted_to_flat_ptr: int, flat_to_sorted_ptr: int,
                    stream: int) -> None:
    """The allocation-free plan: device pointers in, nothing allocated; see the header for
    the size limits and the rule that calls sharing the built-in scratch must not overlap."""
    _check(lib().moe_plan_static(C.c_void_p(topk_ids_ptr), n_tokens, top_k, n_experts,
                                 C.c_void_p(counts_ptr), C.c_void_p(offsets_ptr),
                                 C.c_void_p(sorted_to_flat_ptr), C.c_void_p(flat_to_sorted_ptr),
                                 C.c_void_p(stream)), "moe_plan_static")


def moe_route(logits_ptr: int, n_tokens: int, n_experts: int, top_k: int, ids_ptr: int, w_ptr: int,
              stream: int) -> None:
    _check(lib().moe_route(C.c_void_p(logits_ptr), int(n_tokens), int(n_experts), int(top_k),
                           C.c_void_p(ids_ptr), C.c_void_p(w_ptr), C.c_void_p(stream)), "moe_route")


def route(logits, top_k: int, stream=None):
    """logits: CUDA fp32 tensor [T, E] -> (topk_ids int32 [T, k], topk_w fp32 [T, k])."""
    import torch
    if not (logits.is_cuda and logits.dtype == torch.float32 and logits.dim() == 2 and logits.is_contiguous()):
        raise ValueError("logits must be a contiguous CUDA fp32 [T, E] tensor")
    T, E = logits.shape
    ids = torch.empty((T, top_k), dtype=torch.int32, device=logits.device)
    w = torch.empty((T, top_k), dtype=torch.float32, device=logits.device)
    s = torch.cuda.current_stream(logits.device) if stream is None else stream
    moe_route(logits.data_ptr(), T, E, top_k, ids.data_ptr(), w.data_ptr(), int(s.cuda_stream))
    return ids, w


def moe_sm_count(ctx: int) -> int:
    return int(lib().moe_sm_count(C.c_void_p(ctx)))


def moe_ctas_per_tile(ctx: int) -> int:
    return int(lib().moe_ctas_per_tile(C.c_void_p(ctx)))


# ------------------------------------------------------------------ conveniences

def _ptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


class BoundOp:
    """A moe_op_t plus the tensors it points to (kept alive) and its plan outputs."""

    def __init__(self, c_op: moe_op_t, keep: dict):
        self.c = c_op
        self.t = keep

    def __getattr__(self, name):
        try:
            return self.__dict__["t"][name]
        except KeyError:
            raise AttributeError(name)


def bind_op(cls: int, x, topk_ids, topk_w, w_gate_up, w_down, top_k: int, n_experts: int,
            x_scale=None, s_gate_up=None, s_down=None, ready=None, done=None,
            after_op: int = -1, notify=None, notify_after: int = 0, decode_sms: int = 0) -> BoundOp:
    """Fills a moe_op_t from device tensors and allocates its outputs (y and the plan)."""
    import torch
    T = int(topk_ids.shape[0])
    dev = w_gate_up.device
    H = int(w_down.shape[1])
    y = torch.empty((T, H), dtype=torch.bfloat16, device=dev)
    counts = torch.empty(n_experts, dtype=torch.int32, device=dev)
    offsets = torch.empty(n_experts + 1, dtype=torch.int32, device=dev)
    s2f = torch.empty(max(T * top_k, 1), dtype=torch.int32, device=dev)
    f2s = torch.empty(max(T * top_k, 1), dtype=torch.int32, device=dev)
    keep = dict(x=x, x_scale=x_scale, topk_ids=topk_ids, topk_w=topk_w, w_gate_up=w_gate_up,
                w_down=w_down, s_gate_up=s_gate_up, s_down=s_down, y=y, counts=counts,
                offsets=offsets, sorted_to_flat=s2f, flat_to_sorted=f2s, ready=ready, done=done,
                notify=notify)
    c_op = moe_op_t(cls, T, _ptr(x), _ptr(x_scale), _ptr(topk_ids), _ptr(topk_w),
                    _ptr(w_gate_up), _ptr(w_down), _ptr(s_gate_up), _ptr(s_down), _ptr(y),
                    _ptr(counts), _ptr(offsets), _ptr(s2f), _ptr(f2s), _ptr(ready), _ptr(done),
                    after_op, notify_after, _ptr(notify), decode_sms, MOE_LAYOUT_GATHERED, 0)
    return BoundOp(c_op, keep)


def bind_masked_op(cls: int, x_slabs, counts, w_gate_up, w_down, x_scale=None, s_gate_up=None, s_down=None,
                   ready=None, done=None, after_op: int = -1, decode_sms: int = 0) -> BoundOp:
    """A masked-layout op: x_slabs [E, slab_rows, H] (its scales [E, slab_rows, H/128] for e4m3), counts int32 [E]
    valid rows per slab.  Allocates y in the same slab layout and the offsets output."""
    import torch
    E, slab_rows, H = (int(v) for v in x_slabs.shape)
    dev = w_gate_up.device
    y = torch.zeros((E, slab_rows, H), dtype=torch.bfloat16, device=dev)
    offsets = torch.empty(E + 1, dtype=torch.int32, device=dev)
    keep = dict(x=x_slabs, x_scale=x_scale, w_gate_up=w_gate_up, w_down=w_down, s_gate_up=s_gate_up, s_down=s_down,
                y=y, counts=counts, offsets=offsets, ready=ready, done=done)
    c_op = moe_op_t(cls, 0, _ptr(x_slabs), _ptr(x_scale), None, None, _ptr(w_gate_up), _ptr(w_down), _ptr(s_gate_up),
                    _ptr(s_down), _ptr(y), _ptr(counts), _ptr(offsets), None, None, _ptr(ready), _ptr(done),
                    after_op, 0, None, decode_sms, MOE_LAYOUT_MASKED, slab_rows)
    return BoundOp(c_op, keep)


class Context:
    """Owns the device workspace (a torch uint8 tensor) and the library context."""

    def __init__(self, n_experts: int, top_k: int, hidden: int, inter: int,
                 max_tokens_per_op: int, max_ops: int = 2, dtype: int = MOE_DTYPE_BF16,
                 wait_limit_us: int = 0, tile_log_entries: int = 0, n_ctas: int = 0,
                 device="cuda:0"):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: this library has no CPU path")
        lib()
        self.cfg = moe_config_t(n_experts, top_k, hidden, inter, dtype, max_tokens_per_op,
                                max_ops, wait_limit_us, tile_log_entries, n_ctas)
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        nbytes = moe_workspace_bytes(self.cfg)
        self.workspace = torch.empty(nbytes + 1024, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 1023) // 1024 * 1024
        torch.cuda.synchronize(self.device)
        self.ctx = moe_create(self.cfg, base, nbytes)
        self.workspace_bytes = nbytes

    def close(self):
        if getattr(self, "ctx", None) and moe_destroy is not None:    # None at interpreter shutdown
            moe_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        self.close()

    @staticmethod
    def _stream(stream) -> int:
        import torch
        s = torch.cuda.current_stream() if stream is None else stream
        return int(s.cuda_stream)

    def bind(self, cls, x, topk_ids, topk_w, w_gate_up, w_down, **kw) -> BoundOp:
        return bind_op(cls, x, topk_ids, topk_w, w_gate_up, w_down, self.cfg.top_k,
                       self.cfg.n_experts, **kw)

    def plan(self, slot: int, op: BoundOp, stream=None):
        moe_plan(self.ctx, slot, op.c, self._stream(stream))

    def run(self, slots: Sequence[int], fuse_combine: bool = False, stream=None):
        moe_run(self.ctx, list(slots), fuse_combine, self._stream(stream))

    def plan_pair(self, slot_prefill: int, slot_decode: int, carrier_rows: int = 0, stream=None):
        moe_plan_pair(self.ctx, slot_prefill, slot_decode, carrier_rows, self._stream(stream))

    def run_plain(self, slot: int, stream=None):
        moe_run_plain(self.ctx, slot, self._stream(stream))

    def combine(self, slot: int, stream=None):
        moe_combine(self.ctx, slot, self._stream(stream))

    def set_budget(self, decode_sms: int, stream=None):
        moe_set_budget(self.ctx, decode_sms, self._stream(stream))

    def set_budget_scaled(self, slot: int, q: int, x_moe_star: float, q_max: int, stream=None):
        moe_set_budget_scaled(self.ctx, slot, q, x_moe_star, q_max, self._stream(stream))

    def get_budget(self) -> int:
        return moe_get_budget(self.ctx)

    def status(self):
        return moe_status(self.ctx)

    def check(self):
        """Synchronise and raise if the device recorded an error."""
        import torch
        torch.cuda.synchronize(self.device)
        code, detail = self.status()
        if code != 0:
            raise MoeError(code, f"device status detail={detail}")

    def footprint(self, slot: int):
        return moe_footprint(self.ctx, slot)

    def tile_table(self, slot: int) -> np.ndarray:
        return moe_read_tile_table(self.ctx, slot)

    def tile_log(self) -> np.ndarray:
        return moe_read_tile_log(self.ctx, int(self.cfg.tile_log_entries))

    @property
    def sm_count(self) -> int:
        return moe_sm_count(self.ctx)

    @property
    def ctas_per_tile(self) -> int:
        return moe_ctas_per_tile(self.ctx)
