"""Scheduler properties read from the kernel's tile log: every queue entry runs exactly once,
dependencies are respected, the decode class is served first by the CTAs inside the budget,
and the claim is work conserving (a class with nothing to do lends its CTAs)."""
import numpy as np
import pytest
import torch

import paper_2607_18002_b200 as moe
from workloads import synth

from gpu_util import bind_ops, make_ctx, n_combine_tiles, weights_to

pytestmark = pytest.mark.gpu

# big enough that both classes have work for a while, small enough to run in a second
SPEC = synth.Spec("sched", synth.Shape(32, 4, 1024, 512), ((synth.PREFILL, 4096), (synth.DECODE, 128)),
                  "zipf", 1.0, 1.0, -1.0, 41)


def _run(budget, n_ops=2, n_ctas=0):
    W = weights_to(synth.make_weights(SPEC))
    ops = synth.make_ops(SPEC)[:n_ops]
    ctx = make_ctx(SPEC, max_tokens=4096, max_ops=2, tile_log_entries=1 << 15, n_ctas=n_ctas)
    bound = bind_ops(ctx, ops, W)
    ctx.set_budget(budget)
    for s, b in enumerate(bound):
        ctx.plan(s, b)
    ctx.run(list(range(len(bound))), fuse_combine=True)
    ctx.check()
    return ctx, ctx.tile_log()


def test_every_entry_once_and_dependencies_hold():
    ctx, log = _run(budget=32)
    for slot in (0, 1):
        n = ctx.footprint(slot)[1]
        assert sorted(log["tile"][log["slot"] == slot].tolist()) == list(range(n))
        g = log[log["slot"] == slot]
        first_combine = g["t_claim"][g["kind"] == 2]
        last_gemm = g["t_commit"][g["kind"] < 2].max()
        # a combine tile is published only after the op's last GEMM tile committed; with
        # claim-ahead it may have been *claimed* earlier, so compare commits
        assert g["t_commit"][g["kind"] == 2].min() >= last_gemm
        assert len(first_combine) == n_combine_tiles(SPEC.ops[slot][1])
    assert np.all(log["t_commit"] >= log["t_claim"])


def test_decode_first_inside_the_budget_and_work_conserving():
    q = 32
    ctx, log = _run(budget=q)
    sm = ctx.sm_count
    dec, pre = log[log["cls"] == 0], log[log["cls"] == 1]
    t_dec_end = dec["t_claim"].max()
    # while decode tiles were still being handed out, CTAs inside the budget took only decode
    # tiles (apart from the one tile each may have claimed ahead before decode work appeared)
    inside = log[(log["cta"] < q) & (log["t_claim"] < t_dec_end)]
    assert (inside["cls"] == 1).sum() <= q
    # CTAs outside the budget prefer prefill: they took prefill tiles while both classes had work
    outside = log[(log["cta"] >= q) & (log["t_claim"] < t_dec_end)]
    assert (outside["cls"] == 1).mean() > 0.9
    # work conserving: after the decode queue ran dry, budget CTAs went on with prefill tiles
    late = pre[pre["t_claim"] > t_dec_end]
    units = sm // ctx.ctas_per_tile               # claiming units: CTAs, or pairs of CTAs
    assert len(np.unique(late["cta"][late["cta"] < q])) >= q // ctx.ctas_per_tile // 2
    assert len(np.unique(log["cta"])) == units


def test_decode_op_that_arrives_mid_prefill_is_served_within_the_preemption_bound():
    """Section 4.3: a phase switch happens only at a tile boundary, so a decode operation that
    becomes ready while prefill tiles run is first served after at most the tile a unit executes
    plus the one it had claimed ahead.  The decode op's ready word is the prefill op's notify
    word, set by the kernel itself when a third of the prefill tiles have committed."""
    W = weights_to(synth.make_weights(SPEC))
    ops = synth.make_ops(SPEC)
    ctx = make_ctx(SPEC, max_tokens=4096, max_ops=2, tile_log_entries=1 << 15)
    # reference run: both ops ready at launch
    plain = bind_ops(ctx, ops, W)
    for s, b in enumerate(plain):
        ctx.plan(s, b)
    ctx.run([0, 1], fuse_combine=True)
    ctx.check()
    y_ref = [b.y.clone() for b in plain]
    n_pre = ctx.footprint(0)[1]
    # the same ops, the decode op gated by the prefill op's progress
    word = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    from gpu_util import upload
    d0, d1 = upload(ops[0], None, "cuda:0"), upload(ops[1], None, "cuda:0")
    after = n_pre // 3
    pre = ctx.bind(ops[0].cls, d0["x"], d0["ids"], d0["w"], W.w_gate_up, W.w_down, notify=word, notify_after=after)
    dec = ctx.bind(ops[1].cls, d1["x"], d1["ids"], d1["w"], W.w_gate_up, W.w_down, ready=word)
    ctx.set_budget(32)
    ctx.plan(0, pre)
    ctx.plan(1, dec)
    ctx.run([0, 1], fuse_combine=True)
    ctx.check()
    log = ctx.tile_log()
    assert int(word.item()) == 1
    # results do not depend on when the decode op arrived
    assert torch.equal(pre.y, y_ref[0]) and torch.equal(dec.y, y_ref[1])
    p, d = log[log["cls"] == 1], log[log["cls"] == 0]
    assert len(d) == ctx.footprint(1)[1]
    t_ready = np.sort(p["t_commit"])[after - 1]           # the commit that set the word
    # no decode tile was handed out before the word was set ...
    first = d["t_claim"].min()
    assert first >= t_ready - 2000                        # the log stamp precedes the store by a few hundred ns
    # ... and the first one within two prefill tile times of it
    service = (p["t_commit"].astype(np.int64) - p["t_claim"].astype(np.int64))[p["kind"] < 2]
    assert first - t_ready <= 2 * np.percentile(service, 99)
    # from then on the units inside the budget serve decode tiles
    q_units = 32 // ctx.ctas_per_tile
    t_dec_end = d["t_claim"].max()
    inside = log[(log["cta"] < 32) & (log["t_claim"] > first) & (log["t_claim"] < t_dec_end)]
    assert (inside["cls"] == 1).sum() <= 2 * q_units


def test_one_launch_over_three_layers_with_the_budget_carried_by_the_ops():
    """A kernel that lives across layers (Section 4.2): six operations in one launch, chained by
    after_op (prefill l after prefill l-1, decode l after prefill l-1), every decode op carrying its
    own SM budget.  Results equal the per-layer launches bit for bit."""
    spec = synth.Spec("layers", SPEC.shape, ((synth.PREFILL, 1024), (synth.DECODE, 64)), "zipf", 1.0, 1.0, -1.0, 43,
                      layers=3)
    W = weights_to(synth.make_weights(spec))
    budgets = (16, 32, 64)
    small = make_ctx(spec, max_tokens=1024, max_ops=2)
    y_ref = []
    for l in range(3):
        b = bind_ops(small, synth.make_ops(spec, l), W)
        small.set_budget(budgets[l])
        for s, x in enumerate(b):
            small.plan(s, x)
        small.run([0, 1], fuse_combine=True)
        small.check()
        y_ref.append([x.y.clone() for x in b])
    ctx = make_ctx(spec, max_tokens=1024, max_ops=6, tile_log_entries=1 << 15)
    from gpu_util import upload
    bound = []
    for l in range(3):
        for j, op in enumerate(synth.make_ops(spec, l)):
            d = upload(op, None, "cuda:0")
            bound.append(ctx.bind(op.cls, d["x"], d["ids"], d["w"], W.w_gate_up, W.w_down,
                                  after_op=(2 * (l - 1) if l > 0 else -1),
                                  decode_sms=(budgets[l] if op.cls == synth.DECODE else 0)))
    ctx.set_budget(1)
    for s, b in enumerate(bound):
        ctx.plan(s, b)
    ctx.run(list(range(6)), fuse_combine=True)
    ctx.check()
    for l in range(3):
        assert torch.equal(bound[2 * l].y, y_ref[l][0]) and torch.equal(bound[2 * l + 1].y, y_ref[l][1])
    assert ctx.get_budget() == budgets[2]                 # the last decode op's field was the last write
    log = ctx.tile_log()
    for l in (1, 2):
        done_prev = log["t_commit"][log["slot"] == 2 * (l - 1)].max()
        assert log["t_claim"][log["slot"] == 2 * l].min() >= 0      # claimed ahead is allowed ...
        assert log["t_commit"][log["slot"] == 2 * l].min() >= done_prev     # ... but nothing of it ran before
        assert log["t_commit"][log["slot"] == 2 * l + 1].min() >= done_prev


def test_single_class_uses_all_ctas():
    ctx, log = _run(budget=16, n_ops=1)          # only the prefill op: decode budget must not idle CTAs
    assert len(np.unique(log["cta"])) == ctx.sm_count // ctx.ctas_per_tile
    ctx, log = _run(budget=0, n_ops=2)           # budget 0: decode still gets served (by fallback)
    assert (log["cls"] == 0).sum() == ctx.footprint(1)[1]


def test_scaled_budget_matches_the_formula():
    """moe_set_budget_scaled computes q' of Section 6.4 on the device from the planned footprint."""
    import oracle
    ctx, log = _run(budget=16, n_ops=2)
    x_dec = ctx.footprint(1)[0]                       # slot 1 is the decode op
    c = ctx.ctas_per_tile
    for q, x_star, q_max in ((32, float(x_dec), 148), (32, x_dec / 2.0, 148), (32, x_dec / 7.0, 96),
                             (5, x_dec * 1.5, 148), (0, 10.0, 148), (33, x_dec - 0.5, 148)):
        ctx.set_budget_scaled(1, q, x_star, q_max)
        torch.cuda.synchronize()
        assert ctx.get_budget() == oracle.online_budget(q, x_dec, x_star, q_max, c), (q, x_star, q_max)
    with pytest.raises(moe.MoeError):
        ctx.set_budget_scaled(1, 32, 0.0, 148)


def test_latency_follows_the_footprint_not_the_token_count():
    """Section 6.2: at a fixed token count the kernel time grows with the number of active experts
    (x_moe), and an affine law in x_moe describes it; a small shape keeps this quick."""
    from paper_2607_18002_b200.latency_model import fit_affine, sweep
    rows = sweep(E=64, k=4, H=1024, I=512, tokens=(16, 64), actives=(4, 16, 64), reps=6)
    for T in (16, 64):
        us = [r["us"] for r in rows if r["tokens"] == T]
        assert us[0] < us[-1]                                  # more active experts, same tokens: slower
    assert all(r["x_moe"] == r["active"] for r in rows)        # every active expert holds < 128 rows: one tile each
    alpha, beta, r2 = fit_affine([r["x_moe"] for r in rows], [r["us"] for r in rows])
    assert beta > 0 and r2 > 0.8


def test_sharing_study_runs_and_launch_granularity_sharing_serialises():
    """Two whole-grid launches cannot overlap (one CTA per SM): the decode launch on the high-priority
    stream still ends after the prefill launch, while one persistent launch with a large decode budget
    finishes the decode operation well before the prefill operation (Section 7.3's comparison, small shape)."""
    from paper_2607_18002_b200.sharing_study import study
    rows = study(E=32, k=4, H=1024, I=512, prefill_tokens=8192, decode_tokens=64, budgets=(96,), reps=3)
    by = {(r["arm"], r["q"]): r for r in rows}
    assert all(r["prefill_us"] > 0 and r["decode_us"] > 0 for r in rows if "unavailable" not in r)
    green = [r for r in rows if r["arm"] == "green"]
    assert green and all("unavailable" in r or r["sms_decode"] + r["sms_prefill"] <= 148 for r in green)
    assert by[("streams", None)]["decode_us"] > by[("exclusive", None)]["prefill_us"] * 0.9
    assert by[("apk", 96)]["decode_us"] < by[("apk", 96)]["prefill_us"]


def test_plain_launches_give_the_same_bits_as_the_persistent_kernel():
    """moe_run_plain runs the op's gate/up and down tiles as one plain launch (one claiming unit per queue
    entry, no queue, no budget): the same tile code, so y is bit-identical to the persistent launch; the
    scheduling-overhead study compares the two on a small shape."""
    W = weights_to(synth.make_weights(SPEC))
    ops = synth.make_ops(SPEC)
    ctx = make_ctx(SPEC, max_tokens=4096, max_ops=2, tile_log_entries=1 << 15)
    for s_, op in enumerate(ops):
        b = bind_ops(ctx, [op], W)[0]
        ctx.plan(s_, b)
        ctx.run([s_], fuse_combine=True)
        ctx.check()
        y = b.y.clone()
        b.y.fill_(float("nan"))
        ctx.run_plain(s_)
        ctx.check()
        assert torch.equal(y, b.y)
        log = ctx.tile_log()                   # every GEMM entry exactly once, by the unit with its index
        n_gemm = ctx.footprint(s_)[1] - n_combine_tiles(op.T)
        assert sorted(log["tile"].tolist()) == list(range(n_gemm))
        assert np.array_equal(log["cta"] // 2, log["tile"])
    single = make_ctx(SPEC, max_tokens=4096, max_ops=1, n_ctas=3)          # single-CTA kernel: no plain form
    b = bind_ops(single, ops[1:], W)[0]
    single.plan(0, b)
    with pytest.raises(moe.MoeError):
        single.run_plain(0)
    from paper_2607_18002_b200.sharing_study import scheduler_overhead
    rows = scheduler_overhead(E=32, k=4, H=1024, I=512, prefill_tokens=2048, zipf_s=1.0, decode_tokens=32,
                              actives=(8, 32), reps=3)
    assert len(rows) == 3 and all(r["same_bits"] and r["persistent_us"] > 0 and r["plain_us"] > 0 for r in rows)


def test_a_whole_layer_step_replays_from_a_cuda_graph():
    """Every call of a layer step only enqueues work (a 4-byte budget write, the plan kernels, the pairing, the
    persistent launch), so the step can be captured once and replayed without the host touching it again -- the
    property the paper's kernel is built around (Section 4.2: no CPU reconfiguration between layers).  New routing
    written into the same buffers is picked up by the replay."""
    spec = synth.Spec("graph", SPEC.shape, ((synth.PREFILL, 1500), (synth.DECODE, 48)), "zipf", 1.0, 1.0, -1.0, 45, layers=2)
    W = weights_to(synth.make_weights(spec))
    ctx = make_ctx(spec, max_tokens=1548, max_ops=2)
    ops0, ops1 = synth.make_ops(spec, 0), synth.make_ops(spec, 1)
    bound = bind_ops(ctx, ops0, W)

    def step():
        ctx.set_budget(32)
        ctx.plan(0, bound[0])
        ctx.plan(1, bound[1])
        ctx.plan_pair(0, 1, 0)
        ctx.run([0, 1], fuse_combine=True)

    step()                                     # first calls upload the descriptors: keep them out of the capture
    ctx.check()
    y0 = [b.y.clone() for b in bound]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            step()
    torch.cuda.current_stream().wait_stream(side)
    for b in bound:
        b.y.zero_()
    g.replay()
    ctx.check()
    assert all(torch.equal(a, b.y) for a, b in zip(y0, bound))
    # other inputs in the same buffers: the replay plans and runs them
    from gpu_util import upload
    for b, op in zip(bound, ops1):
        d = upload(op, None, "cuda:0")
        b.x.copy_(d["x"]); b.topk_ids.copy_(d["ids"]); b.topk_w.copy_(d["w"])
    g.replay()
    ctx.check()
    y_graph = [b.y.clone() for b in bound]
    step()
    ctx.check()
    assert all(torch.equal(a, b.y) for a, b in zip(y_graph, bound))
    import oracle
    from gpu_util import assert_close, oracle_weights
    OW = oracle_weights(spec, synth.make_weights(spec))
    for b, op in zip(bound, ops1):
        assert_close(b.y.float().cpu().numpy(), oracle.forward(OW, op.x, None, op.ids, op.w)["y"])
