"""Seeded synthetic inputs for the routed-MoE expert path.

This module only *draws inputs* (activations, expert weights, router outputs).
It holds none of the path's own arithmetic (no histogram, permutation, FFN or
combine) and is imported by the tests, the bench and the smoke check so that the
CPU oracle and the CUDA library consume the same bytes.  It imports neither of
them.

Workloads (shapes follow the paper's evaluation setting of 256 routed experts
with top-8 routing, Section 7.1, and a decode batch of 128 tokens next to a
prefill batch of 8192 tokens, Section 7.3):

  c1  tiny bf16 layer, 48 prefill + 16 decode tokens, softmax -> top-2 router
  c2  decode-only bf16 layer, 128 tokens, uniform top-8 of 256
  c3  prefill-only bf16 layer, 8192 tokens, Zipf(1.2) expert popularity
  c4  mixed stream: per layer 16384 prefill + 256 decode, Zipf(s~U[0.6,1.6])
  c5  FP8 e4m3 block-scaled layer, 4096 prefill + 512 decode, Zipf(1.0)

All tensors are returned as CPU torch tensors in their *stored* dtype (bf16,
or e4m3 bytes plus fp32 scales); routing is numpy int32 / float32.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor
from typing import List, Optional

import numpy as np
import torch

DECODE, PREFILL = 0, 1
E4M3_MAX = 448.0


@dataclasses.dataclass(frozen=True)
class Shape:
    E: int          # routed experts
    k: int          # experts per token
    H: int          # hidden size
    I: int          # expert intermediate size
    dtype: str = "bf16"   # "bf16" | "fp8"


@dataclasses.dataclass
class Weights:
    w_gate_up: torch.Tensor            # [E, 2I, H]  gate rows 0..I-1, up rows I..2I-1
    w_down: torch.Tensor               # [E, H, I]
    s_gate_up: Optional[torch.Tensor] = None   # [E, 2I/128, H/128] fp32 (fp8 only)
    s_down: Optional[torch.Tensor] = None      # [E, H/128, I/128] fp32 (fp8 only)


@dataclasses.dataclass
class Op:
    cls: int                           # DECODE or PREFILL
    x: torch.Tensor                    # [T, H] bf16, or uint8 e4m3 codes
    ids: np.ndarray                    # [T, k] int32, distinct per token
    w: np.ndarray                      # [T, k] float32, sums to 1 per token
    x_scale: Optional[torch.Tensor] = None     # [T, H/128] fp32 (fp8 only)

    @property
    def T(self) -> int:
        return int(self.ids.shape[0])


@dataclasses.dataclass(frozen=True)
class Spec:
    name: str
    shape: Shape
    ops: tuple                 # ((cls, T), ...)
    routing: str               # "softmax_topk" | "uniform" | "zipf"
    zipf_s: Optional[float]    # None -> drawn per layer from U[0.6, 1.6]
    x_std: float
    w_std: float
    seed: int
    layers: int = 1


SPECS = {
    "c1": Spec("c1", Shape(8, 2, 256, 512), ((PREFILL, 48), (DECODE, 16)),
               "softmax_topk", None, 0.02, 0.02, 0),
    # c1 at O(1) output scale, so that an absolute tolerance cannot hide a wrong result
    "c1u": Spec("c1u", Shape(8, 2, 256, 512), ((PREFILL, 48), (DECODE, 16)),
                "softmax_topk", None, 1.0, -1.0, 10),
    "c2": Spec("c2", Shape(256, 8, 3072, 1536), ((DECODE, 128),),
               "uniform", None, 1.0, 0.02, 2),
    "c3": Spec("c3", Shape(256, 8, 3072, 1536), ((PREFILL, 8192),),
               "zipf", 1.2, 1.0, 0.02, 3),
    "c4": Spec("c4", Shape(256, 8, 3072, 1536), ((PREFILL, 16384), (DECODE, 256)),
               "zipf", None, 1.0, 0.02, 4, layers=8),
    "c5": Spec("c5", Shape(256, 8, 6144, 2048, "fp8"), ((PREFILL, 4096), (DECODE, 512)),
               "zipf", 1.0, 1.0, 1.0, 5),
}
# profiling-size variants (same H, I, k and routing law; 64 experts, so that the weights are
# 1.8 GB -- well above L2, small enough for a profiler to save and restore)
SPECS["c2s"] = scaled_ = dataclasses.replace(SPECS["c2"], name="c2s", shape=Shape(64, 8, 3072, 1536),
                                             ops=((DECODE, 32),))
SPECS["c3s"] = dataclasses.replace(SPECS["c3"], name="c3s", shape=Shape(64, 8, 3072, 1536),
                                   ops=((PREFILL, 2048),))
SPECS["c4s"] = dataclasses.replace(SPECS["c4"], name="c4s", shape=Shape(64, 8, 3072, 1536),
                                   ops=((PREFILL, 4096), (DECODE, 64)), layers=2)
SPECS["c5s"] = dataclasses.replace(SPECS["c5"], name="c5s", shape=Shape(32, 8, 6144, 2048, "fp8"),
                                   ops=((PREFILL, 512), (DECODE, 64)))
del scaled_
C4_BUDGETS = (16, 32, 64)     # decode SM budget cycled between layers
C5_BUDGET = 96                # decode SM budget of the single co-scheduled FP8 launch (the config names none)


def scaled(spec: Spec, **kw) -> Spec:
    """A copy of a spec with some fields replaced (smaller test variants)."""
    return dataclasses.replace(spec, **kw)


# --------------------------------------------------------------------------- tensors

def _normal_bf16(out: torch.Tensor, std: float, seed_key) -> None:
    rng = np.random.default_rng(seed_key)
    a = rng.standard_normal(out.numel(), dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    out.copy_(torch.from_numpy(a).view(out.shape))


def _quant_blocks(v: torch.Tensor, br: int, bc: int):
    """fp32 [r, c] -> (e4m3 codes as uint8 [r, c], fp32 scales [r/br, c/bc]).

    scale = amax/448 per (br x bc) block (1 where the block is all zero); the
    stored code is round-to-nearest-even of v * (448/amax), clamped to +-448.
    """
    r, c = v.shape
    blk = v.view(r // br, br, c // bc, bc)
    amax = blk.abs().amax(dim=(1, 3))
    safe = torch.where(amax > 0, amax, torch.full_like(amax, E4M3_MAX))
    scale = (safe / E4M3_MAX).to(torch.float32)
    q = blk * (E4M3_MAX / safe)[:, None, :, None]
    q = q.clamp_(-E4M3_MAX, E4M3_MAX).reshape(r, c).to(torch.float8_e4m3fn)
    return q.view(torch.uint8), scale


def _expert_std(spec: Spec, fan_in: int) -> float:
    return spec.w_std if spec.w_std > 0 else 1.0 / float(np.sqrt(fan_in))


def make_weights(spec: Spec, layer: int = 0, threads: int = 8) -> Weights:
    sh = spec.shape
    E, H, I = sh.E, sh.H, sh.I
    fp8 = sh.dtype == "fp8"
    dt = torch.uint8 if fp8 else torch.bfloat16
    w1 = torch.empty((E, 2 * I, H), dtype=dt)
    w2 = torch.empty((E, H, I), dtype=dt)
    s1 = torch.empty((E, 2 * I // 128, H // 128), dtype=torch.float32) if fp8 else None
    s2 = torch.empty((E, H // 128, I // 128), dtype=torch.float32) if fp8 else None
    std1, std2 = _expert_std(spec, H), _expert_std(spec, I)

    def one(e: int) -> None:
        if fp8:
            for (w, s, shape, std, tag) in ((w1, s1, (2 * I, H), std1, 1), (w2, s2, (H, I), std2, 2)):
                rng = np.random.default_rng([spec.seed, layer, tag, e])
                v = torch.from_numpy(rng.standard_normal(shape, dtype=np.float32))
                if std != 1.0:
                    v *= std
                q, sc = _quant_blocks(v, 128, 128)
                w[e].copy_(q)
                s[e].copy_(sc)
        else:
            _normal_bf16(w1[e], std1, [spec.seed, layer, 1, e])
            _normal_bf16(w2[e], std2, [spec.seed, layer, 2, e])

    with ThreadPoolExecutor(max_workers=max(1, threads)) as pool:
        list(pool.map(one, range(E)))
    return Weights(w1, w2, s1, s2)


def make_x(spec: Spec, T: int, layer: int, op_index: int):
    sh = spec.shape
    rng = np.random.default_rng([spec.seed, layer, 3, op_index])
    v = torch.from_numpy(rng.standard_normal((T, sh.H), dtype=np.float32))
    if spec.x_std != 1.0:
        v *= spec.x_std
    if sh.dtype == "fp8":
        q, sc = _quant_blocks(v, 1, 128)
        return q, sc
    return v.to(torch.bfloat16), None


# --------------------------------------------------------------------------- routing

def _order_slots(ids: np.ndarray, p: np.ndarray):
    """Slot order: descending probability, ties to the lower expert id."""
    order = np.lexsort((ids, -p), axis=1)
    return np.take_along_axis(ids, order, 1), np.take_along_axis(p, order, 1)


def route_softmax_topk(logits: np.ndarray, k: int):
    """softmax over all experts (fp32, max-subtracted) -> k largest -> renormalise."""
    z = logits.astype(np.float32)
    z = z - z.max(axis=1, keepdims=True)
    ez = np.exp(z, dtype=np.float32)
    p = ez / ez.sum(axis=1, keepdims=True, dtype=np.float32)
    E = p.shape[1]
    eid = np.broadcast_to(np.arange(E, dtype=np.int32), p.shape)
    order = np.lexsort((eid, -p), axis=1)[:, :k]
    ids = order.astype(np.int32)
    psel = np.take_along_axis(p, order, 1)
    w = (psel / psel.sum(axis=1, keepdims=True, dtype=np.float32)).astype(np.float32)
    return ids, w


def _weights_over_chosen(rng, ids: np.ndarray):
    z = rng.standard_normal(ids.shape, dtype=np.float32)
    z = z - z.max(axis=1, keepdims=True)
    ez = np.exp(z, dtype=np.float32)
    p = (ez / ez.sum(axis=1, keepdims=True, dtype=np.float32)).astype(np.float32)
    ids, p = _order_slots(ids, p)
    return ids.astype(np.int32), p.astype(np.float32)


def route_popularity(rng, T: int, k: int, log_pi: np.ndarray):
    """k distinct experts per token, drawn by successive sampling proportional to
    pi among the remaining ones (Gumbel-top-k on log pi)."""
    g = rng.gumbel(size=(T, log_pi.shape[0]))
    keys = log_pi[None, :] + g
    ids = np.argpartition(-keys, k - 1, axis=1)[:, :k].astype(np.int32)
    return _weights_over_chosen(rng, ids)


def route_active_pool(rng, T: int, k: int, E: int, n_active: int):
    """k distinct experts per token, uniform over a seeded pool of `n_active` of the E experts:
    the same number of tokens with a chosen number of active experts (the setting of the paper's
    tile-aware latency model, Section 6.2)."""
    if not k <= n_active <= E:
        raise ValueError("need k <= n_active <= E")
    pool = np.sort(rng.permutation(E)[:n_active])
    log_pi = np.full(E, -np.inf)
    log_pi[pool] = 0.0
    g = rng.gumbel(size=(T, E))
    keys = np.where(np.isfinite(log_pi)[None, :], g, -np.inf)
    ids = np.argpartition(-keys, k - 1, axis=1)[:, :k].astype(np.int32)
    return _weights_over_chosen(rng, ids)


def zipf_log_pi(rng, E: int, s: float) -> np.ndarray:
    rank = rng.permutation(E) + 1           # seeded random expert order
    return -s * np.log(rank.astype(np.float64))


def layer_zipf_s(spec: Spec, layer: int) -> float:
    if spec.zipf_s is not None:
        return float(spec.zipf_s)
    return float(np.random.default_rng([spec.seed, layer, 5]).uniform(0.6, 1.6))


def make_routing(spec: Spec, T: int, layer: int, op_index: int):
    sh = spec.shape
    rng = np.random.default_rng([spec.seed, layer, 4, op_index])
    if spec.routing == "softmax_topk":
        logits = rng.standard_normal((T, sh.E), dtype=np.float32)
        return route_softmax_topk(logits, sh.k)
    if spec.routing == "uniform":
        return route_popularity(rng, T, sh.k, np.zeros(sh.E))
    if spec.routing == "zipf":
        # one expert order per layer, shared by the layer's prefill and decode ops
        order_rng = np.random.default_rng([spec.seed, layer, 6])
        log_pi = zipf_log_pi(order_rng, sh.E, layer_zipf_s(spec, layer))
        return route_popularity(rng, T, sh.k, log_pi)
    raise ValueError(spec.routing)


def make_ops(spec: Spec, layer: int = 0) -> List[Op]:
    ops = []
    for i, (cls, T) in enumerate(spec.ops):
        x, xs = make_x(spec, T, layer, i)
        ids, w = make_routing(spec, T, layer, i)
        ops.append(Op(cls, x, ids, w, xs))
    return ops


def adversarial_ids(kind: str, T: int, E: int, k: int, seed: int = 0) -> np.ndarray:
    """Routing patterns that stress the plan step (ids only)."""
    rng = np.random.default_rng([seed, 77])
    if kind == "one_expert":            # every token's slot 0 -> expert E-1; rest distinct
        ids = np.stack([(E - 1 - j) % E for j in range(k)] * T).reshape(T, k)
    elif kind == "two_hot":             # only experts 0 and E-1 ever used (needs k<=2)
        ids = np.tile(np.array([0, E - 1][:k]), (T, 1))
    elif kind == "round_robin":
        ids = (np.arange(T * k).reshape(T, k)) % E
    elif kind == "random":
        ids = np.stack([rng.permutation(E)[:k] for _ in range(T)])
    else:
        raise ValueError(kind)
    return ids.astype(np.int32)
