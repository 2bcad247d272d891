"""The replica timing protocol over gloo with two CPU processes."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2607_18002_b200 import dist as d
    r, w, _ = d.init_from_env("gloo")
    d.barrier()
    mx = d.reduce_scalar(1.0 + r, "max")
    sm = d.reduce_scalar(10.0 * (r + 1), "sum")
    thr = d.job_throughput(100.0, 1.0 + r)          # ranks took 1 s and 2 s for 100 units each
    d.barrier()
    out.put((r, w, mx, sm, thr))
    d.shutdown()


def test_two_rank_reductions():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29000 + os.getpid() % 900
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for r, w, mx, sm, thr in res:
        assert w == 2 and mx == 2.0 and sm == 30.0 and thr == 100.0     # 200 units / 2 s


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    from paper_2607_18002_b200 import dist as d
    assert d.reduce_scalar(3.5, "max") == 3.5 and d.job_throughput(10, 2) == 5.0
