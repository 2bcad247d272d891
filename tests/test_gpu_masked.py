"""The masked decode layout (Section 2.4 of the paper): activations arrive in per-expert slabs [E, slab_rows, H]
with a valid-row count per expert, nothing is permuted, and the expert outputs leave in the same slab layout.
Every valid row must equal the oracle's expert FFN of that row; rows past the count must stay untouched."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_18002_b200 as moe
from workloads import synth

from gpu_util import ATOL8, REL_L2_8, RTOL8, assert_close, make_ctx, oracle_weights, weights_to

pytestmark = pytest.mark.gpu


def _slabs(spec, counts, slab_rows, seed):
    sh = spec.shape
    E = sh.E
    x, xs = synth.make_x(spec, E * slab_rows, 0, seed)              # one seeded row per slab row
    x = x.view(E, slab_rows, sh.H)
    xs = None if xs is None else xs.view(E, slab_rows, sh.H // 128)
    return x, xs


def _run_masked(spec, counts, slab_rows, n_ctas=0, fuse=True):
    sh = spec.shape
    W = synth.make_weights(spec)
    Wd = weights_to(W)
    x, xs = _slabs(spec, counts, slab_rows, 3)
    ctx = make_ctx(spec, max_tokens=-(-sh.E * slab_rows // sh.k), max_ops=1, n_ctas=n_ctas, tile_log_entries=1 << 14)
    cnt = torch.from_numpy(np.asarray(counts, dtype=np.int32)).cuda()
    b = moe.bind_masked_op(moe.MOE_CLASS_DECODE, x.cuda(), cnt, Wd.w_gate_up, Wd.w_down,
                           x_scale=None if xs is None else xs.cuda(), s_gate_up=Wd.s_gate_up, s_down=Wd.s_down)
    b.y.fill_(7.0)
    ctx.plan(0, b)
    ctx.run([0], fuse_combine=fuse)
    ctx.check()
    return ctx, b, W, x, xs


def _check(spec, ctx, b, W, x, xs, counts, slab_rows, fp8=False):
    sh = spec.shape
    counts = np.asarray(counts)
    # plan outputs: offsets are the exclusive scan of the counts, the tile table covers the slabs' valid rows
    assert np.array_equal(b.offsets.cpu().numpy(), np.concatenate([[0], np.cumsum(counts)]).astype(np.int32))
    te, t0, tr = oracle.tiles(counts.astype(np.int32), moe.MOE_TILE_M)
    table = ctx.tile_table(0)
    assert np.array_equal(table[:, 0], te) and np.array_equal(table[:, 2], tr)
    first = np.concatenate([[0], np.cumsum(counts)])[te]           # packed first row of the expert
    assert np.array_equal(table[:, 1], te * slab_rows + (t0 - first))
    rows_e = np.concatenate([np.full(c, e) for e, c in enumerate(counts)]).astype(np.int32)
    rows_r = np.concatenate([np.arange(c) for c in counts]).astype(np.int32)
    flat = rows_e * slab_rows + rows_r
    OW = oracle_weights(spec, W)
    xf = x.reshape(sh.E * slab_rows, sh.H)
    xsf = None if xs is None else xs.reshape(sh.E * slab_rows, sh.H // 128)
    ref = oracle.ffn_rows(OW, xf, xsf, flat, rows_e, round_A=oracle.ROUND_E4M3_1X128 if fp8 else oracle.ROUND_NONE)
    y = b.y.float().cpu().numpy().reshape(sh.E * slab_rows, sh.H)
    if fp8:
        assert_close(y[flat], ref, atol=ATOL8, rtol=RTOL8, rel_l2=REL_L2_8)
    else:
        assert_close(y[flat], ref)
    untouched = np.ones(sh.E * slab_rows, dtype=bool)
    untouched[flat] = False
    assert np.all(y[untouched] == 7.0)                              # rows past a slab's count are not written


@pytest.mark.parametrize("n_ctas", [0, 3], ids=["cta_pairs", "single_ctas"])
def test_masked_decode_matches_oracle(n_ctas):
    spec = synth.Spec("masked", synth.Shape(16, 4, 512, 256), ((synth.DECODE, 1),), "uniform", None, 1.0, -1.0, 51)
    counts = [0, 1, 7, 8, 9, 31, 32, 33, 40, 0, 3, 40, 17, 2, 39, 5]
    slab_rows = 40
    ctx, b, W, x, xs = _run_masked(spec, counts, slab_rows, n_ctas=n_ctas)
    _check(spec, ctx, b, W, x, xs, counts, slab_rows)
    log = ctx.tile_log()
    assert set(np.unique(log["kind"]).tolist()) == {1, 3}           # masked gate/up tiles and down tiles, no combine


@pytest.mark.parametrize("n_ctas", [0, 3], ids=["cta_pairs", "single_ctas"])
def test_masked_slabs_taller_than_a_tile(n_ctas):
    """Slab heights beyond one work tile: counts on and around 64, 128, 256 and 300 rows."""
    spec = synth.Spec("maskedtall", synth.Shape(8, 2, 256, 128), ((synth.PREFILL, 1),), "uniform", None, 1.0, -1.0, 52)
    counts = [63, 64, 65, 128, 129, 256, 257, 300]
    ctx, b, W, x, xs = _run_masked(spec, counts, 300, n_ctas=n_ctas)
    _check(spec, ctx, b, W, x, xs, counts, 300)


def test_masked_fp8_matches_mirrored_oracle():
    spec = synth.Spec("masked8", synth.Shape(8, 2, 512, 256, "fp8"), ((synth.DECODE, 1),), "uniform", None, 1.0, -1.0, 53)
    counts = [5, 0, 16, 33, 1, 128, 129, 140]
    ctx, b, W, x, xs = _run_masked(spec, counts, 140)
    _check(spec, ctx, b, W, x, xs, counts, 140, fp8=True)


def test_masked_rules_and_bad_counts():
    spec = synth.Spec("maskedr", synth.Shape(8, 2, 256, 128), ((synth.DECODE, 1),), "uniform", None, 1.0, -1.0, 54)
    Wd = weights_to(synth.make_weights(spec))
    ctx = make_ctx(spec, max_tokens=64, max_ops=2)                  # scratch rows: 128
    x = torch.zeros(8, 16, 256, dtype=torch.bfloat16, device="cuda")
    cnt = torch.tensor([1, 2, 3, 99, -1, 0, 16, 4], dtype=torch.int32, device="cuda")
    b = moe.bind_masked_op(moe.MOE_CLASS_DECODE, x, cnt, Wd.w_gate_up, Wd.w_down)
    ctx.plan(0, b)
    ctx.run([0], fuse_combine=True)
    torch.cuda.synchronize()
    code, detail = ctx.status()
    assert code == moe.MOE_EBOUNDS and detail[0] == 0 and detail[1] in (3, 4)     # a count the slab cannot hold
    with pytest.raises(moe.MoeError) as ei:                         # nothing to combine in this layout
        ctx.combine(0)
    assert ei.value.code == moe.MOE_EINVAL
    big = torch.zeros(8, 17, 256, dtype=torch.bfloat16, device="cuda")
    bb = moe.bind_masked_op(moe.MOE_CLASS_DECODE, big, cnt, Wd.w_gate_up, Wd.w_down)
    with pytest.raises(moe.MoeError) as ei:                         # 8 * 17 rows > the slot's scratch
        ctx.plan(1, bb)
    assert ei.value.code == moe.MOE_ENOSPC


def test_masked_op_next_to_a_gathered_prefill_op():
    """One launch, two layouts: a masked decode op with priority next to a gathered prefill op."""
    spec = synth.Spec("mix", synth.Shape(16, 4, 512, 256), ((synth.PREFILL, 700),), "zipf", 1.0, 1.0, -1.0, 55)
    W = synth.make_weights(spec)
    Wd = weights_to(W)
    pre = synth.make_ops(spec)[0]
    counts = [3, 0, 9, 1, 4, 12, 0, 2, 7, 7, 1, 0, 5, 16, 2, 8]
    x, _ = _slabs(spec, counts, 16, 4)
    ctx = make_ctx(spec, max_tokens=700, max_ops=2)
    bp = ctx.bind(pre.cls, pre.x.cuda(), torch.from_numpy(pre.ids).cuda(), torch.from_numpy(pre.w).cuda(), Wd.w_gate_up, Wd.w_down)
    bm = moe.bind_masked_op(moe.MOE_CLASS_DECODE, x.cuda(), torch.tensor(counts, dtype=torch.int32, device="cuda"),
                            Wd.w_gate_up, Wd.w_down)
    bm.y.fill_(7.0)
    ctx.set_budget(32)
    ctx.plan(0, bp)
    ctx.plan(1, bm)
    ctx.run([0, 1], fuse_combine=True)
    ctx.check()
    assert_close(bp.y.float().cpu().numpy(), oracle.forward(oracle_weights(spec, W), pre.x, None, pre.ids, pre.w)["y"])

    class _C:                                                       # reuse the slab checker with slot 1
        def tile_table(self, _):
            return ctx.tile_table(1)
    _check(spec, _C(), bm, W, x, None, counts, 16)
