"""How a decode operation fares next to a prefill operation on one GPU under different ways of
sharing it -- the comparison of Section 7.3 of the paper, run on this library's own kernel:

  exclusive   each operation alone on the whole GPU (the floor for both);
  streams     two launches, each with the whole grid, the decode one on a high-priority stream
              right after the prefill one: launch-granularity sharing, no preemption;
  partition   two launches at the same time with disjoint static grids (q CTAs for decode, the
              rest for prefill): what a spatial partition of the SMs gives;
  apk         ONE persistent launch with both operations, tiles claimed from the decode and the
              prefill queue with a decode budget of q CTAs, work conserving.

Times are microseconds from the common start: CUDA events for separate launches; for the single
launch the decode operation's completion comes from the kernel's tile log.

    python -m paper_2607_18002_b200.sharing_study          # prints the table (needs a GPU)
"""
from __future__ import annotations

import json

import numpy as np


def _median(v):
    return float(np.median(np.asarray(v, dtype=np.float64)))


def study(E=256, k=8, H=3072, I=1536, prefill_tokens=16384, decode_tokens=256, budgets=(16, 32, 64, 96),
          reps=5, seed=4, device="cuda:0"):
    import torch

    import paper_2607_18002_b200 as moe
    from workloads import synth

    spec = synth.Spec("sharing", synth.Shape(E, k, H, I), ((synth.PREFILL, prefill_tokens), (synth.DECODE, decode_tokens)),
                      "zipf", 1.0, 0.02, -1.0, seed)
    W = synth.make_weights(spec)
    ops = synth.make_ops(spec)
    dev = torch.device(device)
    w1, w2 = W.w_gate_up.to(dev), W.w_down.to(dev)
    sms = torch.cuda.get_device_properties(dev).multi_processor_count

    def bind(ctx, op):
        return ctx.bind(op.cls, op.x.to(dev), torch.from_numpy(op.ids).to(dev), torch.from_numpy(op.w).to(dev), w1, w2)

    hi = torch.cuda.Stream(device=dev, priority=-1)
    lo = torch.cuda.Stream(device=dev, priority=0)

    def two_launches(n_pre, n_dec):
        """prefill on `lo` with n_pre CTAs, decode on `hi` with n_dec CTAs, released together"""
        cp = moe.Context(E, k, H, I, prefill_tokens, 1, n_ctas=n_pre, device=dev)
        cd = moe.Context(E, k, H, I, decode_tokens, 1, n_ctas=n_dec, device=dev)
        bp, bd = bind(cp, ops[0]), bind(cd, ops[1])
        t_pre, t_dec = [], []
        for _ in range(reps + 1):
            cp.plan(0, bp)
            cd.plan(0, bd)
            torch.cuda.synchronize()
            start = torch.cuda.Event(enable_timing=True)
            ep = torch.cuda.Event(enable_timing=True)
            ed = torch.cuda.Event(enable_timing=True)
            start.record()
            lo.wait_event(start)
            hi.wait_event(start)
            cp.run([0], fuse_combine=True, stream=lo)
            ep.record(lo)
            cd.run([0], fuse_combine=True, stream=hi)
            ed.record(hi)
            torch.cuda.synchronize()
            t_pre.append(1e3 * start.elapsed_time(ep))
            t_dec.append(1e3 * start.elapsed_time(ed))
        cp.check()
        cd.check()
        return _median(t_pre[1:]), _median(t_dec[1:])

    def alone(op, tokens):
        c = moe.Context(E, k, H, I, tokens, 1, device=dev)
        b = bind(c, op)
        ts = []
        for _ in range(reps + 1):
            c.plan(0, b)
            e0 = torch.cuda.Event(enable_timing=True)
            e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
            c.run([0], fuse_combine=True)
            e1.record()
            torch.cuda.synchronize()
            ts.append(1e3 * e0.elapsed_time(e1))
        c.check()
        return _median(ts[1:])

    def apk(q):
        c = moe.Context(E, k, H, I, prefill_tokens, 2, tile_log_entries=1 << 16, device=dev)
        bp, bd = bind(c, ops[0]), bind(c, ops[1])
        t_all, t_dec = [], []
        for _ in range(reps + 1):
            c.set_budget(q)
            c.plan(0, bp)
            c.plan(1, bd)
            e0 = torch.cuda.Event(enable_timing=True)
            e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
            c.run([0, 1], fuse_combine=True)
            e1.record()
            torch.cuda.synchronize()
            log = c.tile_log()
            t0 = log["t_claim"].min()
            t_dec.append((log["t_commit"][log["slot"] == 1].max() - t0) / 1e3)
            t_all.append(1e3 * e0.elapsed_time(e1))
        c.check()
        return _median(t_all[1:]), _median(t_dec[1:])

    rows = []
    p0, d0 = alone(ops[0], prefill_tokens), alone(ops[1], decode_tokens)
    rows.append(dict(arm="exclusive", q=None, prefill_us=p0, decode_us=d0))
    tp, td = two_launches(sms, sms)
    rows.append(dict(arm="streams", q=None, prefill_us=tp, decode_us=td))
    for q in budgets:
        tp, td = two_launches(sms - q, q)
        rows.append(dict(arm="partition", q=q, prefill_us=tp, decode_us=td))
    for q in budgets:
        ta, td = apk(q)
        rows.append(dict(arm="apk", q=q, prefill_us=ta, decode_us=td))
    return rows


def main():
    rows = study()
    for r in rows:
        print("%-10s q=%-4s prefill done %9.1f us   decode done %9.1f us" %
              (r["arm"], "-" if r["q"] is None else r["q"], r["prefill_us"], r["decode_us"]))
    print(json.dumps(rows))


if __name__ == "__main__":
    main()
