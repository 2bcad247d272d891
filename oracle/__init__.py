"""CPU oracle for the routed-MoE expert path -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the bench's CPU-baseline leg may import this
package; the library never does.  It wraps ``moe_oracle.c`` (plain C, double
accumulators, compiled with gcc) through ctypes and composes its steps in the order
the method states them: plan -> per-row expert FFN -> router-weighted combine.

The paper prints no worked numeric example of this path, so numeric parity against
the paper itself is unpinned; every function here is pinned instead against a
closed form, a library routine or brute force in ``tests/test_oracle_pins.py``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moe_oracle.c")
_SO = os.path.join(_HERE, "libmoe_oracle.so")

ROUND_NONE, ROUND_BF16, ROUND_E4M3_1X128 = 0, 1, 2
BF16, E4M3 = 0, 1


def build(force: bool = False) -> str:
    """Compile the C oracle (gcc -O2, OpenMP, no fast-math)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall",
                               "-o", _SO, _SRC, "-lm"])
    return _SO


class _WeightsT(C.Structure):
    _fields_ = [("E", C.c_int), ("k", C.c_int), ("H", C.c_int), ("I", C.c_int),
                ("dtype", C.c_int), ("w_gate_up", C.c_void_p), ("w_down", C.c_void_p),
                ("s_gate_up", C.c_void_p), ("s_down", C.c_void_p)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_e4m3_to_f32.restype = C.c_float
        _lib.orc_e4m3_to_f32.argtypes = [C.c_uint8]
        _lib.orc_f32_to_e4m3.restype = C.c_uint8
        _lib.orc_f32_to_e4m3.argtypes = [C.c_float]
        _lib.orc_bf16_to_f32.restype = C.c_float
        _lib.orc_bf16_to_f32.argtypes = [C.c_uint16]
        _lib.orc_f32_to_bf16.restype = C.c_uint16
        _lib.orc_f32_to_bf16.argtypes = [C.c_float]
        _lib.orc_quant_group.restype = None
    return _lib


def threads() -> int:
    return int(lib().orc_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _np_stored(t):
    """torch tensor (bf16 / uint8 / fp32) or ndarray -> contiguous ndarray view of the bytes."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return np.ascontiguousarray(t)
    import torch
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


# ------------------------------------------------------------------ number formats

def e4m3_to_f32(code: int) -> float:
    return float(lib().orc_e4m3_to_f32(int(code)))


def f32_to_e4m3(v: float) -> int:
    return int(lib().orc_f32_to_e4m3(float(v)))


def bf16_to_f32(b: int) -> float:
    return float(lib().orc_bf16_to_f32(int(b)))


def f32_to_bf16(v: float) -> int:
    return int(lib().orc_f32_to_bf16(float(v)))


def quant_group(v: np.ndarray):
    v = np.ascontiguousarray(v, dtype=np.float32)
    q = np.empty(v.size, dtype=np.uint8)
    s = C.c_float()
    lib().orc_quant_group(_p(v), C.c_int(v.size), _p(q), C.byref(s))
    return q, float(s.value)


# ------------------------------------------------------------------ steps

def router(logits: np.ndarray, k: int):
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    T, E = logits.shape
    ids = np.empty((T, k), dtype=np.int32)
    w = np.empty((T, k), dtype=np.float32)
    rc = lib().orc_router(_p(logits), T, E, k, _p(ids), _p(w))
    if rc:
        raise ValueError(f"orc_router rc={rc}")
    return ids, w


def plan(ids: np.ndarray, E: int):
    """-> counts[E], offsets[E+1], sorted_to_flat[R], flat_to_sorted[R] (int32)."""
    flat = np.ascontiguousarray(ids, dtype=np.int32).reshape(-1)
    R = flat.size
    counts = np.empty(E, dtype=np.int32)
    offsets = np.empty(E + 1, dtype=np.int32)
    s2f = np.empty(R, dtype=np.int32)
    f2s = np.empty(R, dtype=np.int32)
    rc = lib().orc_plan(_p(flat), R, E, _p(counts), _p(offsets), _p(s2f), _p(f2s))
    if rc:
        raise ValueError(f"expert id out of range at flat index {-rc - 1}")
    return counts, offsets, s2f, f2s


def online_budget(q: int, x_moe: int, x_moe_star: float, q_max: int, c: int) -> int:
    """Online SM reallocation (Section 6.4): q' = min(Q_max, ceil_c(q * x_moe / x_moe_star)), where ceil_c rounds
    up to a multiple of the cluster size c."""
    import math
    want = math.ceil(q * x_moe / x_moe_star)
    want = -(-want // c) * c
    return min(q_max, want)


def tiles(counts: np.ndarray, Mt: int):
    """-> (tile_expert, tile_row0, tile_rows); len == x_moe."""
    counts = np.ascontiguousarray(counts, dtype=np.int32)
    E = counts.size
    x = lib().orc_tiles(_p(counts), E, Mt, None, None, None)
    te, t0, tr = (np.empty(x, dtype=np.int32) for _ in range(3))
    lib().orc_tiles(_p(counts), E, Mt, _p(te), _p(t0), _p(tr))
    return te, t0, tr


class Weights:
    """Holds ndarray views of the stored weight bytes and the C descriptor."""

    def __init__(self, E, k, H, I, w_gate_up, w_down, s_gate_up=None, s_down=None):
        self.E, self.k, self.H, self.I = E, k, H, I
        self.w1, self.w2 = _np_stored(w_gate_up), _np_stored(w_down)
        self.s1, self.s2 = _np_stored(s_gate_up), _np_stored(s_down)
        self.dtype = E4M3 if self.w1.dtype == np.uint8 else BF16
        assert self.w1.size == E * 2 * I * H and self.w2.size == E * H * I
        self.c = _WeightsT(E, k, H, I, self.dtype, self.w1.ctypes.data, self.w2.ctypes.data,
                           0 if self.s1 is None else self.s1.ctypes.data,
                           0 if self.s2 is None else self.s2.ctypes.data)


def ffn_rows(W: Weights, x, x_scale, row_token, row_expert, round_A=ROUND_NONE,
             round_D=ROUND_NONE, want_A=False):
    """Expert FFN for routed rows given as (token, expert) pairs -> D [n, H] fp32."""
    xs = _np_stored(x)
    xsc = _np_stored(x_scale)
    rt = np.ascontiguousarray(row_token, dtype=np.int32)
    re = np.ascontiguousarray(row_expert, dtype=np.int32)
    n = rt.size
    D = np.empty((n, W.H), dtype=np.float32)
    A = np.empty((n, W.I), dtype=np.float32) if want_A else None
    rc = lib().orc_ffn_rows(C.byref(W.c), _p(xs), _p(xsc), _p(rt), _p(re), n,
                            int(round_A), int(round_D), _p(D), _p(A))
    if rc:
        raise ValueError(f"orc_ffn_rows rc={rc}")
    return (D, A) if want_A else D


def combine(D: np.ndarray, w: np.ndarray, row_of: np.ndarray, H: int):
    D = np.ascontiguousarray(D, dtype=np.float32)
    w = np.ascontiguousarray(w, dtype=np.float32)
    T, k = w.shape
    row_of = np.ascontiguousarray(row_of, dtype=np.int32).reshape(-1)
    y = np.empty((T, H), dtype=np.float32)
    lib().orc_combine(_p(D), _p(w), _p(row_of), T, k, H, _p(y))
    return y


# ------------------------------------------------------------------ the path, composed

def forward(W: Weights, x, x_scale, ids, w, round_A=ROUND_NONE, round_D=ROUND_NONE):
    """One op through the whole path: plan -> FFN on packed rows -> combine.

    Returns dict(counts, offsets, sorted_to_flat, flat_to_sorted, D, y)."""
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    T, k = ids.shape
    counts, offsets, s2f, f2s = plan(ids, W.E)
    row_token = s2f // k
    row_expert = ids.reshape(-1)[s2f]
    D = ffn_rows(W, x, x_scale, row_token, row_expert, round_A, round_D)
    y = combine(D, w, f2s, W.H)
    return dict(counts=counts, offsets=offsets, sorted_to_flat=s2f, flat_to_sorted=f2s, D=D, y=y)


def forward_tokens(W: Weights, x, x_scale, ids, w, tokens, round_A=ROUND_NONE,
                   round_D=ROUND_NONE):
    """The path restricted to a subset of tokens (the FFN is independent per token,
    Section 2.1): y rows for `tokens`, in the order given."""
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    w = np.ascontiguousarray(w, dtype=np.float32)
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    k = ids.shape[1]
    row_token = np.repeat(tokens, k)
    row_expert = ids[tokens].reshape(-1)
    D = ffn_rows(W, x, x_scale, row_token, row_expert, round_A, round_D)
    ident = np.arange(tokens.size * k, dtype=np.int32)
    return combine(D, w[tokens], ident, W.H)


def dense_token_loop(W: Weights, x, x_scale, ids, w):
    """Brute force, form (i): loop tokens, loop slots, every token through every expert
    it selected; no counts, offsets or permutation involved."""
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    T, k = ids.shape
    y = np.zeros((T, W.H), dtype=np.float64)
    for t in range(T):
        for j in range(k):
            d = ffn_rows(W, x, x_scale, [t], [int(ids[t, j])])[0]
            y[t] += float(w[t, j]) * d.astype(np.float64)
    return y
