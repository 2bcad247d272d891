"""Tile-aware latency model of the expert kernel (Section 6.2 of the paper): the latency of a
decode-sized operation follows its footprint x_moe = sum over active experts of ceil(m_e / M_t)
-- the number of weight tiles it has to stream -- not its token count.

`fit_affine` fits t = alpha + beta * x by least squares; `sweep` measures the persistent kernel
on a GPU for a grid of (tokens, active experts) with seeded synthetic routing and returns the
rows of the paper's "same tokens, different active experts" experiment for this machine.

    python -m paper_2607_18002_b200.latency_model          # prints the table and the fit (needs a GPU)
    python -m paper_2607_18002_b200.latency_model --layouts   # gathered vs masked decode layout (Sections 2.4, 7.4)
"""
from __future__ import annotations

import json

import numpy as np


def fit_affine(x, t):
    """Least-squares alpha, beta of t = alpha + beta * x, and the coefficient of determination."""
    x = np.asarray(x, dtype=np.float64)
    t = np.asarray(t, dtype=np.float64)
    A = np.stack([np.ones_like(x), x], axis=1)
    (alpha, beta), *_ = np.linalg.lstsq(A, t, rcond=None)
    res = t - (alpha + beta * x)
    tot = t - t.mean()
    r2 = 1.0 - float(res @ res) / float(tot @ tot) if float(tot @ tot) > 0 else 1.0
    return float(alpha), float(beta), r2


def sweep(E=256, k=8, H=3072, I=1536, tokens=(32, 128, 512), actives=(8, 16, 32, 64, 128, 256),
          reps=12, seed=7, device="cuda:0"):
    """Kernel time (CUDA events, microseconds, median of `reps` launches after 3 warm-up launches;
    a buffer larger than L2 is written between launches) of one decode op per (tokens, active
    experts).  Returns a list of dicts with tokens, active, x_moe, us."""
    import torch

    import paper_2607_18002_b200 as moe
    from workloads import synth

    spec = synth.Spec("latency_model", synth.Shape(E, k, H, I), ((synth.DECODE, max(tokens)),),
                      "uniform", None, 0.02, -1.0, seed)
    W = synth.make_weights(spec)
    dev = torch.device(device)
    w1, w2 = W.w_gate_up.to(dev), W.w_down.to(dev)
    ctx = moe.Context(E, k, H, I, max(tokens), 1, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    rows = []
    for T in tokens:
        x, _ = synth.make_x(spec, T, 0, 0)
        for A in actives:
            if A < k:
                continue
            rng = np.random.default_rng([seed, T, A])
            ids, w = synth.route_active_pool(rng, T, k, E, A)
            b = ctx.bind(synth.DECODE, x.to(dev), torch.from_numpy(ids).to(dev), torch.from_numpy(w).to(dev), w1, w2)
            ts = []
            for it in range(reps + 3):
                ctx.plan(0, b)
                flush.fill_(it & 1)
                e0 = torch.cuda.Event(enable_timing=True)
                e1 = torch.cuda.Event(enable_timing=True)
                e0.record()
                ctx.run([0], fuse_combine=True)
                e1.record()
                torch.cuda.synchronize()
                ts.append(1e3 * e0.elapsed_time(e1))
            ctx.check()
            rows.append(dict(tokens=T, active=int(len(np.unique(ids))), x_moe=ctx.footprint(0)[0],
                             us=float(np.median(ts[3:]))))
    return rows


def layout_comparison(E=256, k=8, H=3072, I=1536, tokens=128, actives=(8, 16, 32, 64, 128, 256), reps=12, seed=9,
                      device="cuda:0"):
    """The same decode batch through the gathered layout (moe_plan builds the permutation, the kernel gathers token
    rows, the combine returns token order) and through the masked layout of Section 2.4 (the rows already sit in
    per-expert slabs, the plan only scans the counts, rows are loaded as boxes, outputs stay in slabs), over a growing
    number of active experts.  Times are plan + persistent launch in microseconds (CUDA events, median of `reps`, L2
    flushed in between).  Returns rows of dict(active, x_moe, gathered_us, masked_us, slab_rows)."""
    import torch

    import paper_2607_18002_b200 as moe
    from workloads import synth

    spec = synth.Spec("layouts", synth.Shape(E, k, H, I), ((synth.DECODE, tokens),), "uniform", None, 0.02, -1.0, seed)
    W = synth.make_weights(spec)
    dev = torch.device(device)
    w1, w2 = W.w_gate_up.to(dev), W.w_down.to(dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    x, _ = synth.make_x(spec, tokens, 0, 0)

    def timed(ctx, b):
        ts = []
        for it in range(reps + 3):
            flush.fill_(it & 1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            ctx.plan(0, b)
            ctx.run([0], fuse_combine=True)
            e1.record()
            torch.cuda.synchronize()
            ts.append(1e3 * e0.elapsed_time(e1))
        ctx.check()
        return float(np.median(ts[3:]))

    rows = []
    for A in actives:
        if A < k or A > E:
            continue
        ids, w = synth.route_active_pool(np.random.default_rng([seed, A]), tokens, k, E, A)
        counts = np.bincount(ids.reshape(-1), minlength=E).astype(np.int32)
        slab_rows = max(8, -(-int(counts.max()) // 8) * 8)
        ctx = moe.Context(E, k, H, I, max(tokens, -(-E * slab_rows // k)), 1, device=dev)
        bg = ctx.bind(synth.DECODE, x.to(dev), torch.from_numpy(ids).to(dev), torch.from_numpy(w).to(dev), w1, w2)
        t_g = timed(ctx, bg)
        x_moe = ctx.footprint(0)[0]
        # the dispatch the masked layout presumes: token rows copied into their experts' slabs, in routing order
        order = np.argsort(ids.reshape(-1), kind="stable")
        slab = torch.zeros(E, slab_rows, H, dtype=x.dtype)
        rank = np.concatenate([np.arange(c) for c in counts])
        slab[torch.from_numpy(ids.reshape(-1)[order]).long(), torch.from_numpy(rank).long()] = x[torch.from_numpy(order // k).long()]
        bm = moe.bind_masked_op(synth.DECODE, slab.to(dev), torch.from_numpy(counts).to(dev), w1, w2)
        t_m = timed(ctx, bm)
        rows.append(dict(active=int((counts > 0).sum()), x_moe=x_moe, gathered_us=t_g, masked_us=t_m, slab_rows=slab_rows))
        del ctx
    return rows


def main():
    import sys
    if "--layouts" in sys.argv:
        for r in layout_comparison():
            print("active experts %3d  x_moe %3d  gathered %8.1f us  masked %8.1f us  (%+.1f us, slabs of %d rows)" %
                  (r["active"], r["x_moe"], r["gathered_us"], r["masked_us"], r["masked_us"] - r["gathered_us"], r["slab_rows"]))
        return
    rows = sweep()
    alpha, beta, r2 = fit_affine([r["x_moe"] for r in rows], [r["us"] for r in rows])
    for r in rows:
        print("tokens %4d  active experts %3d  x_moe %3d  %8.1f us" % (r["tokens"], r["active"], r["x_moe"], r["us"]))
    print(json.dumps(dict(alpha_us=alpha, beta_us_per_tile=beta, r2=r2, rows=rows)))


if __name__ == "__main__":
    main()
