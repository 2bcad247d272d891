"""Helpers shared by the GPU parity tests: run one spec through the C-ABI library and
through the oracle on the same seeded inputs."""
import numpy as np
import torch

import oracle
import paper_2607_18002_b200 as moe
from workloads import synth

# acceptance tolerances for bf16 with fp32 accumulation (elementwise) and a scale-free check
ATOL, RTOL, REL_L2 = 1e-2, 1e-2, 5e-3
# ... and for the FP8 path, against the oracle that mirrors the on-path quantisation of A
ATOL8, RTOL8, REL_L2_8 = 4e-2, 4e-2, 3e-2


def n_combine_tiles(T: int) -> int:
    """Combine entries of an op's queue list: 16 tokens per tile, 4 for a batch of at most 1024 tokens."""
    ct = 4 if T <= 1024 else 16
    return -(-T // ct)


def upload(op: synth.Op, W: synth.Weights, dev="cuda:0"):
    t = lambda a: None if a is None else (a if isinstance(a, torch.Tensor) else torch.from_numpy(a)).to(dev)
    return dict(x=t(op.x), x_scale=t(op.x_scale), ids=t(op.ids), w=t(op.w))


def make_ctx(spec: synth.Spec, max_tokens=None, max_ops=None, **kw) -> moe.Context:
    sh = spec.shape
    mt = max_tokens or max(T for _, T in spec.ops)
    dtype = moe.MOE_DTYPE_FP8_E4M3 if sh.dtype == "fp8" else moe.MOE_DTYPE_BF16
    return moe.Context(sh.E, sh.k, sh.H, sh.I, mt, max_ops or len(spec.ops), dtype=dtype, **kw)


def bind_ops(ctx, ops, Wd, dev="cuda:0", **kw):
    bound = []
    for op in ops:
        d = upload(op, None, dev)
        bound.append(ctx.bind(op.cls, d["x"], d["ids"], d["w"], Wd.w_gate_up, Wd.w_down,
                              x_scale=d["x_scale"], s_gate_up=Wd.s_gate_up, s_down=Wd.s_down, **kw))
    return bound


def weights_to(W: synth.Weights, dev="cuda:0") -> synth.Weights:
    t = lambda a: None if a is None else a.to(dev)
    return synth.Weights(t(W.w_gate_up), t(W.w_down), t(W.s_gate_up), t(W.s_down))


def oracle_weights(spec: synth.Spec, W: synth.Weights) -> oracle.Weights:
    sh = spec.shape
    return oracle.Weights(sh.E, sh.k, sh.H, sh.I, W.w_gate_up, W.w_down, W.s_gate_up, W.s_down)


def check_plan(bound, op: synth.Op, E: int):
    counts, offsets, s2f, f2s = oracle.plan(op.ids, E)
    R = op.ids.size
    assert np.array_equal(bound.counts.cpu().numpy(), counts)
    assert np.array_equal(bound.offsets.cpu().numpy(), offsets)
    assert np.array_equal(bound.sorted_to_flat.cpu().numpy()[:R], s2f)
    assert np.array_equal(bound.flat_to_sorted.cpu().numpy()[:R], f2s)
    return counts


def check_tiles(ctx, slot, counts):
    te, t0, tr = oracle.tiles(counts, moe.MOE_TILE_M)
    table = ctx.tile_table(slot)
    x_moe, _ = ctx.footprint(slot)
    assert x_moe == len(te)
    assert np.array_equal(table[:, 0], te) and np.array_equal(table[:, 1], t0)
    assert np.array_equal(table[:, 2], tr)


def assert_close(y_gpu: np.ndarray, y_ref: np.ndarray, atol=ATOL, rtol=RTOL, rel_l2=REL_L2):
    y_gpu = y_gpu.astype(np.float64)
    y_ref = y_ref.astype(np.float64)
    assert np.all(np.isfinite(y_gpu))
    err = np.abs(y_gpu - y_ref)
    bad = err > atol + rtol * np.abs(y_ref)
    assert not bad.any(), f"{bad.sum()} elements outside tolerance, max err {err.max():.4g}"
    rel = np.linalg.norm(y_gpu - y_ref) / max(np.linalg.norm(y_ref), 1e-30)
    assert rel <= rel_l2, f"relative L2 error {rel:.3e} > {rel_l2}"
    return rel
