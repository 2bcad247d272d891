"""The paired form of a decode + prefill op (moe_plan_pair): decode rows ride in carrier tiles together with
prefill rows of the same expert, so a launch streams each weight tile once for both ops.  A row's arithmetic
does not depend on its tile, so outputs must equal the unpaired launch bit for bit, and the oracle within the
usual tolerance; the plan's public outputs must not change."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_18002_b200 as moe
from workloads import synth

from gpu_util import (ATOL8, REL_L2_8, RTOL8, assert_close, bind_ops, check_plan, check_tiles, make_ctx,
                      oracle_weights, weights_to)

pytestmark = pytest.mark.gpu

SMALL = synth.Spec("small", synth.Shape(8, 2, 256, 128), ((synth.PREFILL, 300), (synth.DECODE, 37)),
                   "softmax_topk", None, 1.0, -1.0, 21)


def _both_ways(spec, ops, W, carrier_rows, fuse, budget=8, **ctx_kw):
    """Runs the two ops unpaired and paired in one context; returns (ctx, bound, y_unpaired, log_paired)."""
    Wd = weights_to(W)
    total = sum(o.T for o in ops)
    ctx = make_ctx(spec, max_tokens=total, max_ops=2, tile_log_entries=1 << 15, **ctx_kw)
    bound = bind_ops(ctx, ops, Wd)
    ctx.set_budget(budget)

    def run(pair):
        for b in bound:
            b.y.fill_(float("nan"))
        for s, b in enumerate(bound):
            ctx.plan(s, b)
        if pair:
            ctx.plan_pair(0, 1, carrier_rows)
        ctx.run([0, 1], fuse_combine=fuse)
        if not fuse:
            ctx.combine(0)
            ctx.combine(1)
        ctx.check()
        return [b.y.clone() for b in bound]

    y_plain = run(False)
    n_plain = len(ctx.tile_log())
    y_pair = run(True)
    log = ctx.tile_log()
    for a, b in zip(y_plain, y_pair):
        assert torch.equal(a, b)
    assert len(log) <= n_plain                       # pairing never adds queue entries
    for s in (0, 1):                                 # each list's entries exactly once
        t = np.sort(log["tile"][log["slot"] == s])
        assert np.array_equal(t, np.arange(len(t)))
    return ctx, bound, y_plain, log


@pytest.mark.parametrize("fuse", [False, True])
@pytest.mark.parametrize("carrier_rows", [128, 256])
@pytest.mark.parametrize("n_ctas", [0, 3], ids=["cta_pairs", "single_ctas"])
def test_paired_launch_equals_unpaired_launch_and_oracle(n_ctas, carrier_rows, fuse):
    spec = SMALL
    W = synth.make_weights(spec)
    ops = synth.make_ops(spec)
    ctx, bound, y, log = _both_ways(spec, ops, W, carrier_rows, fuse, n_ctas=n_ctas)
    OW = oracle_weights(spec, W)
    for s, (b, op) in enumerate(zip(bound, ops)):
        counts = check_plan(b, op, spec.shape.E)             # the public plan outputs are untouched
        check_tiles(ctx, s, counts)
        assert_close(b.y.float().cpu().numpy(), oracle.forward(OW, op.x, None, op.ids, op.w)["y"])
    # decode rows were carried: the decode list has GEMM entries, and fewer entries ran than unpaired
    assert ((log["slot"] == 1) & (log["kind"] < 2)).sum() > 0


def test_paired_row_counts_around_the_carrier_capacity():
    """Per expert (prefill rows, decode rows) on and around what one carrier tile holds, an expert with decode rows
    only, one with prefill rows only, one with neither, and decode rows that need more than one tile."""
    combos = [(0, 5), (300, 0), (0, 0), (1, 1), (100, 8), (120, 8), (121, 8), (128, 8), (250, 6), (256, 1), (300, 127),
              (300, 128), (300, 129), (40, 300), (513, 64), (5, 123)]
    E, k, H, I = len(combos), 1, 512, 256
    rng = np.random.default_rng(19)
    ids_p = np.concatenate([np.full(cp, e) for e, (cp, _) in enumerate(combos)]).astype(np.int32)
    ids_d = np.concatenate([np.full(cd, e) for e, (_, cd) in enumerate(combos)]).astype(np.int32)
    ids_p, ids_d = ids_p[rng.permutation(ids_p.size)].reshape(-1, 1), ids_d[rng.permutation(ids_d.size)].reshape(-1, 1)
    spec = synth.Spec("cap", synth.Shape(E, k, H, I), ((synth.PREFILL, ids_p.shape[0]), (synth.DECODE, ids_d.shape[0])),
                      "uniform", None, 1.0, -1.0, 37)
    W = synth.make_weights(spec)
    ops = []
    for i, (cls, ids) in enumerate(((synth.PREFILL, ids_p), (synth.DECODE, ids_d))):
        x, _ = synth.make_x(spec, ids.shape[0], 0, i)
        ops.append(synth.Op(cls, x, ids, np.ones(ids.shape, np.float32)))
    OW = oracle_weights(spec, W)
    refs = [oracle.forward(OW, op.x, None, op.ids, op.w)["y"] for op in ops]
    for carrier_rows in (128, 256):
        for n_ctas in (0, 3):
            ctx, bound, _, _ = _both_ways(spec, ops, W, carrier_rows, True, n_ctas=n_ctas)
            for b, op, ref in zip(bound, ops, refs):
                check_plan(b, op, E)
                assert_close(b.y.float().cpu().numpy(), ref)


def test_pairing_rules():
    spec = SMALL
    W = synth.make_weights(spec)
    Wd = weights_to(W)
    ops = synth.make_ops(spec)
    ctx = make_ctx(spec, max_tokens=337, max_ops=3)
    bound = bind_ops(ctx, ops, Wd)
    with pytest.raises(moe.MoeError) as ei:                 # nothing planned yet
        ctx.plan_pair(0, 1)
    assert ei.value.code == moe.MOE_ENOTPLANNED
    ctx.plan(0, bound[0])
    ctx.plan(1, bound[1])
    for args in ((1, 0, 0), (0, 0, 0), (0, 1, 64), (0, 5, 0)):     # classes swapped, same slot, bad height, bad slot
        with pytest.raises(moe.MoeError) as ei:
            ctx.plan_pair(*args)
        assert ei.value.code == moe.MOE_EINVAL
    # other weights: no tile can serve both ops
    W2 = weights_to(synth.make_weights(synth.scaled(spec, seed=99)))
    other = bind_ops(ctx, ops[1:], W2)[0]
    ctx.plan(2, other)
    with pytest.raises(moe.MoeError) as ei:
        ctx.plan_pair(0, 2)
    assert ei.value.code == moe.MOE_EINVAL
    # the shared row space must fit one slot's scratch
    tight = make_ctx(spec, max_tokens=300, max_ops=2)
    tb = bind_ops(tight, ops, Wd)
    tight.plan(0, tb[0])
    tight.plan(1, tb[1])
    with pytest.raises(moe.MoeError) as ei:
        tight.plan_pair(0, 1)
    assert ei.value.code == moe.MOE_ENOSPC
    # paired, then only one of the two in a launch: the plain form runs; a new plan ends the pairing
    ctx.plan_pair(0, 1)
    ctx.run([0, 1], fuse_combine=True)
    ctx.check()
    y = [b.y.clone() for b in bound]
    bound[1].y.zero_()
    ctx.run([1], fuse_combine=True)
    ctx.check()
    assert torch.equal(bound[1].y, y[1])
    ctx.plan(1, bound[1])
    bound[0].y.zero_()
    bound[1].y.zero_()
    ctx.run([0, 1], fuse_combine=True)
    ctx.check()
    assert torch.equal(bound[0].y, y[0]) and torch.equal(bound[1].y, y[1])


def test_paired_ops_with_done_words_and_a_successor():
    """The prefill op of a pair is complete only when the decode op's carrier tiles are; an op chained after it
    starts after that, and both done words are set."""
    spec = synth.Spec("chainp", SMALL.shape, ((synth.PREFILL, 300), (synth.DECODE, 37), (synth.PREFILL, 90)),
                      "softmax_topk", None, 1.0, -1.0, 24)
    W = synth.make_weights(spec)
    Wd = weights_to(W)
    ops = synth.make_ops(spec)
    ctx = make_ctx(spec, max_tokens=337, max_ops=3, tile_log_entries=1 << 14)
    done = torch.zeros(3, dtype=torch.int32, device="cuda")
    b0 = bind_ops(ctx, ops[0:1], Wd, done=done[0:1])[0]
    b1 = bind_ops(ctx, ops[1:2], Wd, done=done[1:2])[0]
    b2 = bind_ops(ctx, ops[2:3], Wd, done=done[2:3], after_op=0)[0]
    for s, b in enumerate((b0, b1, b2)):
        ctx.plan(s, b)
    ctx.plan_pair(0, 1, 128)
    ctx.set_budget(0)
    ctx.run([0, 1, 2], fuse_combine=True)
    ctx.check()
    assert done.tolist() == [1, 1, 1]
    log = ctx.tile_log()
    carriers = log[(log["slot"] == 1) & (log["kind"] < 2)]
    assert log["t_commit"][log["slot"] == 2].min() >= carriers["t_commit"].max()
    assert log["t_commit"][log["slot"] == 2].min() >= log["t_commit"][log["slot"] == 0].max()
    OW = oracle_weights(spec, W)
    for b, op in zip((b0, b1, b2), ops):
        assert_close(b.y.float().cpu().numpy(), oracle.forward(OW, op.x, None, op.ids, op.w)["y"])


@pytest.mark.parametrize("shape", [synth.Shape(8, 2, 512, 256, "fp8"), synth.Shape(16, 4, 768, 384, "fp8")], ids=["h512", "h768"])
def test_paired_fp8_equals_unpaired_and_mirrored_oracle(shape):
    spec = synth.Spec("fp8p", shape, ((synth.PREFILL, 300), (synth.DECODE, 37)), "softmax_topk", None, 1.0, -1.0, 35)
    W = synth.make_weights(spec)
    ops = synth.make_ops(spec)
    OW = oracle_weights(spec, W)
    for carrier_rows in (128, 256):                   # 256: the carrier runs as two 128-row tiles
        ctx, bound, _, _ = _both_ways(spec, ops, W, carrier_rows, True)
        for b, op in zip(bound, ops):
            check_plan(b, op, shape.E)
            ref = oracle.forward(OW, op.x, op.x_scale, op.ids, op.w, round_A=oracle.ROUND_E4M3_1X128)
            assert_close(b.y.float().cpu().numpy(), ref["y"], atol=ATOL8, rtol=RTOL8, rel_l2=REL_L2_8)


def test_paired_seeded_random_shapes():
    rng = np.random.default_rng(4242)
    for i in range(6):
        E = int(rng.integers(2, 41))
        k = int(rng.integers(1, min(E, 8) + 1))
        H, I = int(rng.choice([256, 512, 768])), int(rng.choice([128, 256, 384]))
        T1, T0 = int(rng.integers(1, 900)), int(rng.integers(1, 80))
        spec = synth.Spec("randp", synth.Shape(E, k, H, I), ((synth.PREFILL, T1), (synth.DECODE, T0)), "zipf", 1.1, 1.0,
                          -1.0, 300 + i)
        W = synth.make_weights(spec)
        ops = synth.make_ops(spec)
        ctx, bound, _, _ = _both_ways(spec, ops, W, int(rng.choice([128, 256])), bool(rng.integers(0, 2)),
                                      budget=int(rng.integers(0, 64)), n_ctas=int(rng.choice([0, 0, 5, 8])))
        OW = oracle_weights(spec, W)
        for b, op in zip(bound, ops):
            check_plan(b, op, E)
            assert_close(b.y.float().cpu().numpy(), oracle.forward(OW, op.x, None, op.ids, op.w)["y"])


def test_poisoned_scratch_changes_nothing(monkeypatch):
    """With MOE_APK_POISON=1 the scratch rows start every launch as NaN patterns: outputs stay bit-identical (every row
    that is read was written by the same launch), unpaired, paired and in e4m3."""
    for shape in (SMALL.shape, synth.Shape(8, 2, 512, 256, "fp8")):
        spec = synth.scaled(SMALL, shape=shape)
        W = synth.make_weights(spec)
        ops = synth.make_ops(spec)
        monkeypatch.delenv("MOE_APK_POISON", raising=False)
        _, _, y_ref, _ = _both_ways(spec, ops, W, 128, True)
        monkeypatch.setenv("MOE_APK_POISON", "1")
        _, bound, y, _ = _both_ways(spec, ops, W, 128, True)
        for a, b in zip(y_ref, y):
            assert torch.equal(a, b) and torch.isfinite(b.float()).all()


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_three_paired_layers_in_one_launch(dtype):
    """Six operations in one launch, chained by after_op (prefill l and decode l after prefill l-1), the two ops of
    every layer paired: results equal the per-layer unpaired launches bit for bit."""
    shape = synth.Shape(32, 4, 1024, 512, dtype)
    spec = synth.Spec("layersp", shape, ((synth.PREFILL, 1024), (synth.DECODE, 64)), "zipf", 1.0, 1.0, -1.0, 43, layers=3)
    W = weights_to(synth.make_weights(spec))
    small = make_ctx(spec, max_tokens=1024, max_ops=2)
    y_ref = []
    for l in range(3):
        b = bind_ops(small, synth.make_ops(spec, l), W)
        for s_, x in enumerate(b):
            small.plan(s_, x)
        small.run([0, 1], fuse_combine=True)
        small.check()
        y_ref.append([x.y.clone() for x in b])
    ctx = make_ctx(spec, max_tokens=1024 + 64, max_ops=6, tile_log_entries=1 << 15)
    from gpu_util import upload
    bound = []
    for l in range(3):
        for op in synth.make_ops(spec, l):
            d = upload(op, None, "cuda:0")
            bound.append(ctx.bind(op.cls, d["x"], d["ids"], d["w"], W.w_gate_up, W.w_down, x_scale=d["x_scale"],
                                  s_gate_up=W.s_gate_up, s_down=W.s_down,
                                  after_op=(2 * (l - 1) if l > 0 else -1),
                                  decode_sms=((16, 32, 64)[l] if op.cls == synth.DECODE else 0)))
    for s_, b in enumerate(bound):
        ctx.plan(s_, b)
    for l in range(3):
        ctx.plan_pair(2 * l, 2 * l + 1, 128 if dtype == "fp8" else (128, 256, 0)[l])
    ctx.run(list(range(6)), fuse_combine=True)
    ctx.check()
    for l in range(3):
        assert torch.equal(bound[2 * l].y, y_ref[l][0]) and torch.equal(bound[2 * l + 1].y, y_ref[l][1])
    log = ctx.tile_log()
    for l in (1, 2):
        done_prev = log["t_commit"][log["slot"] == 2 * (l - 1)].max()
        assert log["t_commit"][log["slot"] == 2 * l].min() >= done_prev
        assert log["t_commit"][log["slot"] == 2 * l + 1].min() >= done_prev
