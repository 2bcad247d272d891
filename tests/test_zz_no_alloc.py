"""moe_plan_static -- the plan entry point that allocates nothing -- against moe_plan.

Collected last on purpose: a failure here must not keep any other test from running.
The entry point keeps its scratch in a fixed device array inside the library, so it serves
callers that cannot allocate device memory themselves (their memory belongs to another
allocator, or they may not make calls that can synchronise the device).  The test calls it
through the C ABI twice in a row, on different inputs, and requires the same counts,
offsets and permutation as the context-based moe_plan, bit for bit (integer outputs: the
tolerance of the other plan tests is exact equality)."""
import numpy as np
import pytest
import torch

import paper_2607_18002_b200 as moe
from workloads import synth

pytestmark = pytest.mark.gpu


def _plan_with_context(ids_dev, T, E, k):
    spec = synth.Spec("na", synth.Shape(E, k, 256, 128), ((synth.PREFILL, T),), "uniform", None,
                      1.0, -1.0, 3)
    W = synth.make_weights(spec)
    ctx = moe.Context(E, k, 256, 128, T, max_ops=1)
    b = ctx.bind(synth.PREFILL, torch.zeros(T, 256, dtype=torch.bfloat16, device="cuda"), ids_dev,
                 torch.full((T, k), 1.0 / k, device="cuda"), W.w_gate_up.cuda(), W.w_down.cuda())
    ctx.plan(0, b)
    ctx.check()
    return b


def _plan_static(ids_dev, T, E, k):
    out = [torch.full((n,), -7, dtype=torch.int32, device="cuda") for n in (E, E + 1, T * k, T * k)]
    stream = torch.cuda.current_stream().cuda_stream
    moe.moe_plan_static(ids_dev.data_ptr(), T, k, E, *(o.data_ptr() for o in out), stream)
    torch.cuda.synchronize()
    return out


def test_two_calls_in_a_row_match_moe_plan():
    for T, E, k, seed in ((4096, 256, 8, 1), (777, 64, 6, 2)):     # second call: smaller, other shape
        ids = synth.make_routing(synth.scaled(synth.SPECS["c3"], shape=synth.Shape(E, k, 256, 128),
                                              seed=seed), T, 0, 0)[0]
        ids_dev = torch.from_numpy(ids).cuda()
        want = _plan_with_context(ids_dev, T, E, k)
        counts, offsets, s2f, f2s = _plan_static(ids_dev, T, E, k)
        assert torch.equal(counts, want.counts) and torch.equal(offsets, want.offsets)
        assert torch.equal(s2f, want.sorted_to_flat[:T * k])
        assert torch.equal(f2s, want.flat_to_sorted[:T * k])
        assert np.array_equal(s2f.cpu().numpy(), np.argsort(ids.reshape(-1), kind="stable"))


def test_sizes_beyond_the_fixed_scratch_are_refused():
    d = torch.zeros(8, dtype=torch.int32, device="cuda")
    for T, k, E in ((moe.MOE_PLAN_STATIC_MAX_ROWS // 8 + 1, 8, 256), (16, 2, 257)):
        with pytest.raises(moe.MoeError) as ei:
            moe.moe_plan_static(d.data_ptr(), T, k, E, d.data_ptr(), d.data_ptr(), d.data_ptr(),
                                d.data_ptr(), 0)
        assert ei.value.code == moe.MOE_ENOSPC
    # the largest size that fits still works
    T, k, E = moe.MOE_PLAN_STATIC_MAX_ROWS // 8, 8, 256
    ids = synth.adversarial_ids("random", T, E, k, 9)
    counts, offsets, s2f, f2s = _plan_static(torch.from_numpy(ids).cuda(), T, E, k)
    assert np.array_equal(s2f.cpu().numpy(), np.argsort(ids.reshape(-1), kind="stable"))
    assert int(offsets[-1]) == T * k
