"""How a decode operation fares next to a prefill operation on one GPU under different ways of
sharing it -- the comparison of Section 7.3 of the paper, run on this library's own kernel:

  exclusive   each operation alone on the whole GPU (the floor for both);
  streams     two launches, each with the whole grid, the decode one on a high-priority stream
              right after the prefill one: launch-granularity sharing, no preemption;
  partition   two launches at the same time with disjoint static grids (q CTAs for decode, the
              rest for prefill): what a spatial partition of the SMs gives;
  green       the same two launches, each on a stream of its own CUDA green context whose SM set the
              driver enforces (q SMs for decode, the remaining SMs for prefill); left out with the
              driver's answer if green contexts cannot be made here;
  apk         ONE persistent launch with both operations, tiles claimed from the decode and the
              prefill queue with a decode budget of q CTAs, work conserving;
  apk_paired  the same launch with the two operations paired (moe_plan_pair): an expert's decode rows
              travel in carrier tiles of up to 128 / 256 rows together with prefill rows of that expert.

Times are microseconds from the common start: CUDA events for separate launches; for the single
launch the decode operation's completion comes from the kernel's tile log.

    python -m paper_2607_18002_b200.sharing_study          # prints the table (needs a GPU)

`scheduler_overhead` is the companion experiment of Section 7.4: the persistent kernel against plain
launches of the same tile code, on a prefill-sized op and on decode-sized ops over 8..256 active experts.

    python -m paper_2607_18002_b200.sharing_study --overhead
    python -m paper_2607_18002_b200.sharing_study --few-experts     # 8 192 prefill + 128 decode tokens on 8 experts
"""
from __future__ import annotations

import json

import numpy as np


def _median(v):
    return float(np.median(np.asarray(v, dtype=np.float64)))


def study(E=256, k=8, H=3072, I=1536, prefill_tokens=16384, decode_tokens=256, budgets=(16, 32, 64, 96, 112, 128),
          reps=5, seed=4, device="cuda:0", decode_active=None):
    """decode_active: None routes the decode tokens by the same Zipf law as the prefill tokens (they then touch
    most experts); a number confines them to a seeded pool of that many experts -- the regime of the paper's
    experiment, where a decode batch meets few active experts on each GPU."""
    import torch

    import paper_2607_18002_b200 as moe
    from workloads import synth

    spec = synth.Spec("sharing", synth.Shape(E, k, H, I), ((synth.PREFILL, prefill_tokens), (synth.DECODE, decode_tokens)),
                      "zipf", 1.0, 0.02, -1.0, seed)
    W = synth.make_weights(spec)
    ops = synth.make_ops(spec)
    if decode_active is not None:
        ids, w = synth.route_active_pool(np.random.default_rng([seed, 8]), decode_tokens, k, E, decode_active)
        ops[1] = synth.Op(ops[1].cls, ops[1].x, ids, w, ops[1].x_scale)
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

    def green_launches(q):
        """Two green contexts that split the SMs (q for decode, the rest for prefill), one stream in each, the two
        single-op launches released together.  Returns (prefill_us, decode_us, sms_decode, sms_prefill), or a string
        saying why the driver would not make the contexts."""
        try:
            from cuda.bindings import driver as cu
        except Exception as e:                      # pragma: no cover
            return f"cuda-python not importable: {e}"
        made = []
        try:
            err, cdev = cu.cuDeviceGet(dev.index or 0)
            if err != cu.CUresult.CUDA_SUCCESS:
                return f"cuDeviceGet: {err}"
            err, res = cu.cuDeviceGetDevResource(cdev, cu.CUdevResourceType.CU_DEV_RESOURCE_TYPE_SM)
            if err != cu.CUresult.CUDA_SUCCESS:
                return f"cuDeviceGetDevResource: {err}"
            err, groups, n_groups, rest = cu.cuDevSmResourceSplitByCount(1, res, 0, q)
            if err != cu.CUresult.CUDA_SUCCESS or n_groups < 1:
                return f"cuDevSmResourceSplitByCount: {err}"
            streams, counts = [], []
            for r in (groups[0], rest):
                err, desc = cu.cuDevResourceGenerateDesc([r], 1)
                if err != cu.CUresult.CUDA_SUCCESS:
                    return f"cuDevResourceGenerateDesc: {err}"
                err, g = cu.cuGreenCtxCreate(desc, cdev, cu.CUgreenCtxCreate_flags.CU_GREEN_CTX_DEFAULT_STREAM)
                if err != cu.CUresult.CUDA_SUCCESS:
                    return f"cuGreenCtxCreate: {err}"
                made.append(g)
                err, st = cu.cuGreenCtxStreamCreate(g, cu.CUstream_flags.CU_STREAM_NON_BLOCKING, 0)
                if err != cu.CUresult.CUDA_SUCCESS:
                    return f"cuGreenCtxStreamCreate: {err}"
                streams.append(st)
                counts.append(int(r.sm.smCount))
            s_dec, s_pre = (torch.cuda.ExternalStream(int(st), device=dev) for st in streams)
            n_dec, n_pre = counts[0] // 2 * 2, counts[1] // 2 * 2
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
                s_pre.wait_event(start)
                s_dec.wait_event(start)
                cp.run([0], fuse_combine=True, stream=s_pre)
                ep.record(s_pre)
                cd.run([0], fuse_combine=True, stream=s_dec)
                ed.record(s_dec)
                torch.cuda.synchronize()
                t_pre.append(1e3 * start.elapsed_time(ep))
                t_dec.append(1e3 * start.elapsed_time(ed))
            cp.check()
            cd.check()
            for st in streams:
                cu.cuStreamDestroy(st)
            return _median(t_pre[1:]), _median(t_dec[1:]), counts[0], counts[1]
        except Exception as e:
            return f"{type(e).__name__}: {e}"
        finally:
            torch.cuda.synchronize()
            for g in made:
                cu.cuGreenCtxDestroy(g)

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

    def apk(q, carrier_rows=None):
        c = moe.Context(E, k, H, I, prefill_tokens + decode_tokens, 2, tile_log_entries=1 << 16, device=dev)
        bp, bd = bind(c, ops[0]), bind(c, ops[1])
        t_all, t_dec = [], []
        for _ in range(reps + 1):
            c.set_budget(q)
            c.plan(0, bp)
            c.plan(1, bd)
            if carrier_rows:
                c.plan_pair(0, 1, carrier_rows)
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
        got = green_launches(q)
        if isinstance(got, str):
            rows.append(dict(arm="green", q=q, prefill_us=float("nan"), decode_us=float("nan"), unavailable=got))
            break
        rows.append(dict(arm="green", q=q, prefill_us=got[0], decode_us=got[1], sms_decode=got[2], sms_prefill=got[3]))
    for q in budgets:
        ta, td = apk(q)
        rows.append(dict(arm="apk", q=q, prefill_us=ta, decode_us=td))
    for cr in (128, 256):
        for q in budgets:
            ta, td = apk(q, cr)
            rows.append(dict(arm=f"apk_paired{cr}", q=q, prefill_us=ta, decode_us=td))
    return rows


def scheduler_overhead(E=256, k=8, H=3072, I=1536, prefill_tokens=8192, zipf_s=1.2, decode_tokens=128,
                       actives=(8, 32, 128, 256), reps=10, seed=3, device="cuda:0"):
    """What the persistent kernel's tile scheduling costs against plain launches of the SAME tile code
    (the experiment of Section 7.4): for a prefill-sized op (contiguous layout, Zipf routing) and for a
    decode-sized op over a growing number of active experts, the time of moe_run + moe_combine next to the
    time of moe_run_plain (one launch with a claiming unit per tile, then the combine).  CUDA events, median of `reps` after one warm-up, L2 flushed between launches.  Returns rows of
    dict(case, x_moe, persistent_us, plain_us)."""
    import torch

    import paper_2607_18002_b200 as moe
    from workloads import synth

    dev = torch.device(device)
    spec = synth.Spec("overhead", synth.Shape(E, k, H, I), ((synth.PREFILL, prefill_tokens),), "zipf", zipf_s, 1.0, 0.02, seed)
    W = synth.make_weights(spec)
    w1, w2 = W.w_gate_up.to(dev), W.w_down.to(dev)
    ctx = moe.Context(E, k, H, I, max(prefill_tokens, decode_tokens), 1, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def timed(b, plain):
        ts = []
        for it in range(reps + 1):
            ctx.plan(0, b)
            flush.fill_(it & 1)
            torch.cuda.synchronize()                # run_plain reads the tile count: keep that wait out of the timing
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            if plain:
                ctx.run_plain(0)
            else:
                ctx.run([0], fuse_combine=False)
                ctx.combine(0)
            e1.record()
            torch.cuda.synchronize()
            ts.append(1e3 * e0.elapsed_time(e1))
        ctx.check()
        return _median(ts[1:])

    rows = []
    op = synth.make_ops(spec)[0]
    b = ctx.bind(op.cls, op.x.to(dev), torch.from_numpy(op.ids).to(dev), torch.from_numpy(op.w).to(dev), w1, w2)
    t_pers, y = timed(b, False), b.y.clone()
    t_plain = timed(b, True)
    rows.append(dict(case=f"prefill {prefill_tokens} tokens", x_moe=ctx.footprint(0)[0], persistent_us=t_pers, plain_us=t_plain,
                     same_bits=bool(torch.equal(y, b.y))))
    x, _ = synth.make_x(spec, decode_tokens, 0, 1)
    for A in actives:
        if A < k or A > E:
            continue
        ids, w = synth.route_active_pool(np.random.default_rng([seed, A]), decode_tokens, k, E, A)
        b = ctx.bind(synth.DECODE, x.to(dev), torch.from_numpy(ids).to(dev), torch.from_numpy(w).to(dev), w1, w2)
        t_pers, y = timed(b, False), b.y.clone()
        t_plain = timed(b, True)
        rows.append(dict(case=f"decode {decode_tokens} tokens, {A} active experts", x_moe=ctx.footprint(0)[0],
                         persistent_us=t_pers, plain_us=t_plain, same_bits=bool(torch.equal(y, b.y))))
    return rows


def main():
    import sys
    if "--overhead" in sys.argv:
        rows = scheduler_overhead()
        for r in rows:
            print("%-42s x_moe %4d  persistent %8.1f us  plain launches %8.1f us  (%+.1f %%, %+.1f us)" %
                  (r["case"], r["x_moe"], r["persistent_us"], r["plain_us"],
                   100.0 * (r["persistent_us"] / r["plain_us"] - 1.0), r["persistent_us"] - r["plain_us"]))
        print(json.dumps(rows))
        return
    if "--few-experts" in sys.argv:      # the paper's setting: 8 192 prefill tokens next to 128 decode tokens on 8 experts
        rows = study(prefill_tokens=8192, decode_tokens=128, decode_active=8, budgets=(16, 32, 64, 96, 128), reps=7)
    else:
        rows = study()
    for r in rows:
        print("%-13s q=%-4s prefill done %9.1f us   decode done %9.1f us  %s" %
              (r["arm"], "-" if r["q"] is None else r["q"], r["prefill_us"], r["decode_us"],
               r.get("unavailable", "") or ("SMs %d + %d" % (r["sms_decode"], r["sms_prefill"]) if "sms_decode" in r else "")))
    print(json.dumps(rows))


if __name__ == "__main__":
    main()
