"""The GPU router against the oracle's router (softmax over all experts in fp32, the k largest
probabilities with ties to the lower expert id, weights renormalised over the chosen k)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_18002_b200 as moe
from workloads import synth

from gpu_util import bind_ops, make_ctx, weights_to, assert_close, oracle_weights

pytestmark = pytest.mark.gpu


def _check(logits: np.ndarray, k: int, min_same: float = 0.999):
    ids_ref, w_ref = oracle.router(logits, k)
    ids, w = moe.route(torch.from_numpy(logits).cuda(), k)
    torch.cuda.synchronize()
    ids, w = ids.cpu().numpy(), w.cpu().numpy()
    same = (ids == ids_ref).all(axis=1)
    # Where the picks differ the logits must tie at that point: the oracle compares fp32
    # probabilities, the kernel the logits themselves, and exp() can map two different logits to
    # one probability.  Both picks are then valid; everything else must agree exactly.
    for t in np.nonzero(~same)[0]:
        z = logits[t].astype(np.float64)
        p = np.exp(z - z.max()).astype(np.float32)
        assert sorted(p[ids[t]].tolist()) == sorted(p[ids_ref[t]].tolist()), t
        assert len(set(ids[t].tolist())) == k
    assert same.mean() >= min_same
    np.testing.assert_allclose(w[same], w_ref[same], rtol=2e-6, atol=1e-8)
    np.testing.assert_allclose(w.sum(axis=1), 1.0, rtol=0, atol=1e-6)
    assert ((ids >= 0) & (ids < logits.shape[1])).all()
    return ids, w


@pytest.mark.parametrize("T,E,k", [(64, 8, 2), (4096, 256, 8), (1000, 40, 5), (33, 1024, 32), (7, 5, 5), (129, 64, 1)])
def test_router_matches_oracle(T, E, k):
    rng = np.random.default_rng([T, E, k])
    _check(rng.standard_normal((T, E), dtype=np.float32), k)


def test_router_ties_and_extreme_logits():
    rng = np.random.default_rng(5)
    T, E, k = 257, 96, 8
    z = rng.integers(-3, 4, size=(T, E)).astype(np.float32)          # many exact ties
    ids, _ = _check(z, k)
    ids_ref, _ = oracle.router(z, k)
    assert (ids == ids_ref).all()                                     # equal logits: equal probabilities, same tie rule
    z = (rng.standard_normal((T, E)) * 40).astype(np.float32)        # probabilities underflow far from the maximum
    z[:, 0] = 80.0
    _check(z, k, min_same=0.9)                                       # underflowed probabilities tie at 0: several valid picks
    z = np.zeros((T, E), dtype=np.float32)                            # all equal: experts 0..k-1 in order
    ids, w = _check(z, k)
    assert (ids == np.arange(k)[None, :]).all() and np.allclose(w, 1.0 / k)


def test_router_argument_checks():
    z = torch.zeros((4, 8), dtype=torch.float32, device="cuda")
    with pytest.raises(moe.MoeError):
        moe.route(z, 9)                                               # k > E
    with pytest.raises(moe.MoeError):
        moe.route(torch.zeros((4, 2048), dtype=torch.float32, device="cuda"), 2)
    ids, w = moe.route(torch.zeros((0, 8), dtype=torch.float32, device="cuda"), 2)
    assert ids.shape == (0, 2) and w.shape == (0, 2)


def test_route_plan_run_end_to_end():
    """logits -> moe_route -> moe_plan -> moe_run on the device, against the oracle's own chain."""
    spec = synth.Spec("routed", synth.Shape(16, 4, 512, 256), ((synth.PREFILL, 200),), "softmax_topk", None, 1.0, -1.0, 9)
    W = synth.make_weights(spec)
    x, _ = synth.make_x(spec, 200, 0, 0)
    logits = np.random.default_rng(12).standard_normal((200, 16), dtype=np.float32)
    ids_ref, w_ref = oracle.router(logits, 4)
    ids, w = moe.route(torch.from_numpy(logits).cuda(), 4)
    assert (ids.cpu().numpy() == ids_ref).all()
    ctx = make_ctx(spec)
    Wd = weights_to(W)
    b = ctx.bind(synth.PREFILL, x.cuda(), ids, w, Wd.w_gate_up, Wd.w_down)
    ctx.plan(0, b)
    ctx.run([0], fuse_combine=True)
    ctx.check()
    ref = oracle.forward(oracle_weights(spec, W), x, None, ids_ref, w_ref)
    assert_close(b.y.float().cpu().numpy(), ref["y"])
