"""Pins for the CPU oracle: each of its steps is checked against something other than
itself -- a library routine, a closed form, brute force, or an invariant -- chosen so a
dropped term, a wrong index or a transposed operand fails at least one test."""
import numpy as np
import pytest
import torch

import oracle
from workloads import synth


def _tiny_weights(E, H, I, seed, std=None):
    g = torch.Generator().manual_seed(seed)
    w1 = (torch.randn(E, 2 * I, H, generator=g) * (std or H ** -0.5)).to(torch.bfloat16)
    w2 = (torch.randn(E, H, I, generator=g) * (std or I ** -0.5)).to(torch.bfloat16)
    return w1, w2


def _dense_f64(x, w1, w2, ids, w, E):
    """Fully dense float64 evaluation with library matmuls: every token through every
    expert, weighted by the E-wide scatter of the router weights."""
    x = x.to(torch.float64)
    T = x.shape[0]
    I = w2.shape[2]
    m = torch.zeros(T, E, dtype=torch.float64)
    for t in range(T):
        for j in range(ids.shape[1]):
            m[t, ids[t, j]] += float(w[t, j])
    y = torch.zeros(T, x.shape[1], dtype=torch.float64)
    for e in range(E):
        Wg = w1[e, :I].to(torch.float64).T      # [H, I]
        Wu = w1[e, I:].to(torch.float64).T
        Wd = w2[e].to(torch.float64).T          # [I, H]
        a = torch.nn.functional.silu(x @ Wg) * (x @ Wu)
        y += m[:, e:e + 1] * (a @ Wd)
    return y.numpy()


# ------------------------------------------------------------------ plan

@pytest.mark.parametrize("T,E,k,seed", [(5, 3, 2, 0), (64, 8, 2, 1), (128, 256, 8, 2),
                                        (1, 4, 1, 3), (333, 17, 5, 4), (2048, 256, 8, 5)])
def test_plan_equals_stable_argsort(T, E, k, seed):
    ids = synth.adversarial_ids("random", T, E, k, seed)
    counts, offsets, s2f, f2s = oracle.plan(ids, E)
    flat = ids.reshape(-1)
    assert np.array_equal(s2f, np.argsort(flat, kind="stable").astype(np.int32))
    assert np.array_equal(counts, np.bincount(flat, minlength=E))
    assert np.array_equal(offsets, np.concatenate([[0], np.cumsum(counts)]))


@pytest.mark.parametrize("kind,T,E,k", [("one_expert", 37, 8, 2), ("two_hot", 50, 16, 2),
                                        ("round_robin", 129, 7, 3), ("random", 9, 256, 8)])
def test_plan_invariants_and_bruteforce(kind, T, E, k):
    ids = synth.adversarial_ids(kind, T, E, k)
    counts, offsets, s2f, f2s = oracle.plan(ids, E)
    R, flat = T * k, ids.reshape(-1)
    assert counts.sum() == R and offsets[0] == 0 and offsets[E] == R
    assert np.all(np.diff(offsets) >= 0)
    assert np.array_equal(np.sort(s2f), np.arange(R))              # bijection
    assert np.array_equal(f2s[s2f], np.arange(R))                  # inverse
    for e in range(E):
        seg = s2f[offsets[e]:offsets[e + 1]]
        assert np.all(flat[seg] == e)
        assert np.all(np.diff(seg) > 0)                            # stable => unique
        # brute force: rescan all rows for this expert
        assert list(seg) == [i for i in range(R) if flat[i] == e]


def test_plan_rejects_bad_id():
    with pytest.raises(ValueError):
        oracle.plan(np.array([[0, 9]], dtype=np.int32), 8)


@pytest.mark.parametrize("Mt", [16, 32, 64, 128])
def test_tiles_closed_form(Mt):
    rng = np.random.default_rng(Mt)
    counts = rng.integers(0, 700, size=64).astype(np.int32)
    counts[[3, 10]] = 0
    counts[5], counts[6], counts[7] = Mt, Mt + 1, Mt - 1
    te, t0, tr = oracle.tiles(counts, Mt)
    x_moe = sum(-(-int(c) // Mt) for c in counts if c > 0)        # Section 6.2 footprint
    assert len(te) == x_moe
    assert tr.sum() == counts.sum() and tr.min() >= 1 and tr.max() <= Mt
    offsets = np.concatenate([[0], np.cumsum(counts)])
    covered = np.zeros(counts.sum(), dtype=np.int32)
    for e, r0, n in zip(te, t0, tr):
        assert offsets[e] <= r0 and r0 + n <= offsets[e + 1]
        covered[r0:r0 + n] += 1
    assert np.all(covered == 1)                                    # disjoint and covering
    assert np.all(np.diff(te) >= 0)


# ------------------------------------------------------------------ router

def test_router_against_full_sort_and_generator():
    rng = np.random.default_rng(0)
    logits = rng.standard_normal((64, 8)).astype(np.float32)
    ids, w = oracle.router(logits, 2)
    p = torch.softmax(torch.from_numpy(logits).double(), dim=1).numpy()
    order = np.argsort(-p, axis=1, kind="stable")[:, :2]
    assert np.array_equal(ids, order)
    ref_w = np.take_along_axis(p, order, 1)
    ref_w /= ref_w.sum(1, keepdims=True)
    assert np.allclose(w, ref_w, rtol=1e-5, atol=1e-7)
    assert np.allclose(w.sum(1), 1.0, atol=1e-6)
    assert np.all(ids[:, 0] != ids[:, 1])
    gids, gw = synth.route_softmax_topk(logits, 2)                 # the generator's own router
    assert np.array_equal(gids, ids) and np.allclose(gw, w, rtol=1e-5)


def test_router_tie_goes_to_lower_expert():
    logits = np.zeros((1, 6), dtype=np.float32)
    ids, w = oracle.router(logits, 3)
    assert list(ids[0]) == [0, 1, 2] and np.allclose(w, 1 / 3)


# ------------------------------------------------------------------ FFN

def test_ffn_is_dense_swiglu_mlp_for_one_expert():
    H, I, T = 128, 384, 7                     # H != I so a transposed weight cannot pass
    w1, w2 = _tiny_weights(1, H, I, 0)
    x = torch.randn(T, H, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    W = oracle.Weights(1, 1, H, I, w1, w2)
    D, A = oracle.ffn_rows(W, x, None, np.arange(T), np.zeros(T), want_A=True)
    xd = x.double()
    a_ref = torch.nn.functional.silu(xd @ w1[0, :I].double().T) * (xd @ w1[0, I:].double().T)
    d_ref = a_ref @ w2[0].double().T
    assert np.allclose(A, a_ref.numpy(), rtol=2e-6, atol=1e-7)
    assert np.allclose(D, d_ref.numpy(), rtol=1e-5, atol=1e-6)
    # gate and up are not interchangeable: swapping them must change the answer
    a_sw = torch.nn.functional.silu(xd @ w1[0, I:].double().T) * (xd @ w1[0, :I].double().T)
    assert not np.allclose(A, a_sw.numpy(), rtol=1e-3, atol=1e-4)


def test_ffn_special_cases():
    H, I = 128, 128
    w1, w2 = _tiny_weights(2, H, I, 3)
    x = torch.randn(3, H, generator=torch.Generator().manual_seed(4)).to(torch.bfloat16)
    W0 = oracle.Weights(2, 1, H, I, w1, torch.zeros_like(w2))
    assert np.all(oracle.ffn_rows(W0, x, None, [0, 1, 2], [0, 1, 0]) == 0)     # W_down = 0
    assert np.all(oracle.ffn_rows(oracle.Weights(2, 1, H, I, w1, w2),
                                  torch.zeros_like(x), None, [0], [1]) == 0)   # silu(0) = 0
    # silu limits through the FFN: gate = +-c*h-sum, up = 1, down = identity-like
    w1s = torch.zeros(1, 2 * I, H)
    w1s[0, :I, 0] = 1.0           # gate_c = x[0]
    w1s[0, I:, 1] = 1.0           # up_c   = x[1]
    w2s = torch.eye(H, I).unsqueeze(0)
    Ws = oracle.Weights(1, 1, H, I, w1s.to(torch.bfloat16), w2s.to(torch.bfloat16))
    for g, want in ((96.0, 96.0), (-96.0, 0.0), (0.0, 0.0)):
        xs = torch.zeros(1, H)
        xs[0, 0], xs[0, 1] = g, 1.0
        d = oracle.ffn_rows(Ws, xs.to(torch.bfloat16), None, [0], [0])
        assert np.all(np.isfinite(d)) and abs(d[0, 0] - want) < 1e-6


# ------------------------------------------------------------------ combine

def test_combine_applies_each_weight_once():
    T, k, H = 9, 3, 128
    rng = np.random.default_rng(0)
    w = rng.random((T, k)).astype(np.float32)
    w /= w.sum(1, keepdims=True)
    perm = rng.permutation(T * k).astype(np.int32)
    assert np.allclose(oracle.combine(np.ones((T * k, H), np.float32), w, perm, H), 1.0, atol=1e-6)
    # tagged rows: D[p,:] = p, so y[t] = sum_j w[t,j] * perm[t*k+j]
    D = np.repeat(np.arange(T * k, dtype=np.float32)[:, None], H, 1)
    y = oracle.combine(D, w, perm, H)
    want = (w.astype(np.float64) * perm.reshape(T, k)).sum(1)
    assert np.allclose(y[:, 0], want, rtol=1e-6) and np.allclose(y, y[:, :1])
    # linear in w
    y2 = oracle.combine(D, 2 * w, perm, H)
    assert np.allclose(y2, 2 * y, rtol=1e-6)


# ------------------------------------------------------------------ the whole path

@pytest.mark.parametrize("T,E,k,H,I,seed", [(5, 3, 2, 128, 128, 0), (12, 4, 3, 128, 256, 1),
                                            (16, 8, 2, 256, 128, 2)])
def test_forward_equals_dense_evaluation(T, E, k, H, I, seed):
    w1, w2 = _tiny_weights(E, H, I, seed)
    x = torch.randn(T, H, generator=torch.Generator().manual_seed(seed + 9)).to(torch.bfloat16)
    logits = np.random.default_rng(seed).standard_normal((T, E)).astype(np.float32)
    ids, w = oracle.router(logits, k)
    W = oracle.Weights(E, k, H, I, w1, w2)
    out = oracle.forward(W, x, None, ids, w)
    y_dense = _dense_f64(x, w1, w2, ids, w, E)                    # library float64, no plan
    scale = np.abs(y_dense).max()
    assert np.abs(out["y"] - y_dense).max() <= 2e-6 * scale
    y_loop = oracle.dense_token_loop(W, x, None, ids, w)           # token loop, no plan
    assert np.abs(out["y"] - y_loop).max() <= 1e-6 * scale
    # per-token independence: any token alone gives the same row
    sub = np.array([T - 1, 0, T // 2], dtype=np.int32)
    assert np.array_equal(oracle.forward_tokens(W, x, None, ids, w, sub), out["y"][sub])
    # token-permutation equivariance
    perm = np.random.default_rng(7).permutation(T)
    out_p = oracle.forward(W, x[torch.from_numpy(perm)], None, ids[perm], w[perm])
    assert np.array_equal(out_p["y"], out["y"][perm])


def test_c1_config_matches_dense_and_class_split_is_invisible():
    spec = synth.SPECS["c1u"]
    sh = spec.shape
    Wt = synth.make_weights(spec)
    ops = synth.make_ops(spec)
    W = oracle.Weights(sh.E, sh.k, sh.H, sh.I, Wt.w_gate_up, Wt.w_down)
    x = torch.cat([o.x for o in ops])
    ids = np.concatenate([o.ids for o in ops])
    w = np.concatenate([o.w for o in ops])
    whole = oracle.forward(W, x, None, ids, w)["y"]
    parts = np.concatenate([oracle.forward(W, o.x, None, o.ids, o.w)["y"] for o in ops])
    assert np.array_equal(whole, parts)           # one 64-token op == prefill op + decode op
    y_dense = _dense_f64(x, Wt.w_gate_up, Wt.w_down, ids, w, sh.E)
    assert np.abs(whole - y_dense).max() <= 2e-6 * np.abs(y_dense).max()
    assert np.abs(y_dense).mean() > 0.05          # O(1) outputs: the check is not vacuous


# ------------------------------------------------------------------ number formats

def test_e4m3_decode_all_codes_against_library():
    codes = torch.arange(256, dtype=torch.uint8)
    ref = codes.view(torch.float8_e4m3fn).to(torch.float32).numpy()
    got = np.array([oracle.e4m3_to_f32(c) for c in range(256)], dtype=np.float32)
    assert np.array_equal(np.isnan(ref), np.isnan(got))
    ok = ~np.isnan(ref)
    assert np.array_equal(ref[ok], got[ok])
    assert oracle.e4m3_to_f32(0x7e) == 448.0


def test_e4m3_encode_roundtrip_saturation_and_rounding():
    for c in range(256):
        v = oracle.e4m3_to_f32(c)
        if np.isnan(v):
            continue
        back = oracle.f32_to_e4m3(v)
        assert back == c or (v == 0.0 and back in (0x00, 0x80))
    assert oracle.f32_to_e4m3(1e9) == 0x7e and oracle.f32_to_e4m3(-1e9) == 0xfe
    assert oracle.f32_to_e4m3(449.0) == 0x7e and oracle.f32_to_e4m3(464.0) == 0x7e
    # round to nearest even against the library conversion on in-range values
    rng = np.random.default_rng(0)
    v = np.concatenate([rng.uniform(-448, 448, 4000), rng.normal(0, 1, 4000),
                        rng.normal(0, 0.01, 2000)]).astype(np.float32)
    pos = np.array([oracle.e4m3_to_f32(c) for c in range(0x7f)], dtype=np.float64)
    mid = ((pos[1:] + pos[:-1]) / 2).astype(np.float32)            # exact ties
    v = np.concatenate([v, mid, -mid])
    ref = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([oracle.f32_to_e4m3(float(a)) for a in v], dtype=np.uint8)
    same = (ref == got) | ((v == 0) & ((ref | 0x80) == (got | 0x80)))
    assert np.all(same)


def test_quant_group_properties():
    rng = np.random.default_rng(1)
    v = rng.standard_normal(128).astype(np.float32) * 3
    q, s = oracle.quant_group(v)
    deq = np.array([oracle.e4m3_to_f32(c) for c in q], dtype=np.float32) * np.float32(s)
    assert s * 448.0 >= np.abs(v).max() * (1 - 1e-6)
    assert np.abs(deq - v).max() <= np.abs(v).max() * 2 ** -4      # half an ulp at the top binade
    assert np.abs(deq).max() == pytest.approx(np.abs(v).max(), rel=1e-6)   # amax is exact
    q2, s2 = oracle.quant_group(deq)                               # idempotent
    assert np.array_equal(q, q2) and s2 == pytest.approx(s, rel=1e-6)
    q0, s0 = oracle.quant_group(np.zeros(128, np.float32))
    assert s0 == 1.0 and not q0.any()


def test_bf16_conversions_against_library():
    rng = np.random.default_rng(2)
    v = np.concatenate([rng.standard_normal(3000), [0.0, 1.0, 1.00390625, 1.01171875, 3e38, 1e-40]])
    v = v.astype(np.float32)
    ref = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.f32_to_bf16(float(a)) for a in v], dtype=np.uint16)
    assert np.array_equal(ref, got)
    back = np.array([oracle.bf16_to_f32(int(b)) for b in got], dtype=np.float32)
    assert np.array_equal(back, torch.from_numpy(v).to(torch.bfloat16).float().numpy())


def test_fp8_path_equals_dense_on_dequantised_inputs():
    """With e4m3 inputs the oracle must consume code*scale exactly: compare against a
    float64 library evaluation of the dequantised tensors (no intermediate rounding)."""
    spec = synth.scaled(synth.SPECS["c5"], shape=synth.Shape(4, 2, 256, 128, "fp8"),
                        ops=((synth.PREFILL, 6),))
    sh = spec.shape
    Wt = synth.make_weights(spec, threads=2)
    op = synth.make_ops(spec)[0]

    def deq(q, s, br, bc):
        v = q.view(torch.float8_e4m3fn).to(torch.float64)
        return v * s.to(torch.float64).repeat_interleave(br, -2).repeat_interleave(bc, -1)

    w1 = deq(Wt.w_gate_up, Wt.s_gate_up, 128, 128)
    w2 = deq(Wt.w_down, Wt.s_down, 128, 128)
    x = deq(op.x, op.x_scale, 1, 128)
    W = oracle.Weights(sh.E, sh.k, sh.H, sh.I, Wt.w_gate_up, Wt.w_down, Wt.s_gate_up, Wt.s_down)
    out = oracle.forward(W, op.x, op.x_scale, op.ids, op.w)
    y_dense = _dense_f64(x, w1, w2, op.ids, op.w, sh.E)
    assert np.abs(out["y"] - y_dense).max() <= 3e-6 * np.abs(y_dense).max()
    # mirrored on-path quantisation of A changes the result by about e4m3's rounding, not more
    out_q = oracle.forward(W, op.x, op.x_scale, op.ids, op.w, round_A=oracle.ROUND_E4M3_1X128)
    rel = np.linalg.norm(out_q["y"] - out["y"]) / np.linalg.norm(out["y"])
    assert 1e-3 < rel < 6e-2


def _deq_blocks(q, s, br, bc):
    v = q.view(torch.float8_e4m3fn).to(torch.float64)
    return v * s.to(torch.float64).repeat_interleave(br, -2).repeat_interleave(bc, -1)


def _quant_rows_torch(A: torch.Tensor, group: int) -> torch.Tensor:
    """Library restatement of the on-path quantisation: per row and per `group` consecutive columns one
    fp32 scale amax/448 (1 for an all-zero group), codes by torch's float8_e4m3fn cast of v * (448/amax),
    returned dequantised (code * scale) in float64."""
    n, I = A.shape
    blk = A.to(torch.float32).view(n, I // group, group)
    amax = blk.abs().amax(dim=2, keepdim=True)
    scale = torch.where(amax > 0, amax / np.float32(448.0), torch.ones_like(amax))
    inv = torch.where(amax > 0, np.float32(448.0) / amax, torch.zeros_like(amax))
    codes = (blk * inv).clamp(-448.0, 448.0).to(torch.float8_e4m3fn)
    return (codes.to(torch.float32) * scale).view(n, I).to(torch.float64)


@pytest.mark.parametrize("I", [256, 384])
def test_mirrored_e4m3_rounding_of_the_intermediate_is_per_row_per_128_columns(I):
    """The one quantisation on the FP8 path: the SwiGLU output goes to e4m3 with one fp32 scale per row and
    per 128 consecutive columns (scale = amax/448) BEFORE the down projection.  With two or three groups per
    row, the oracle's rounded result must equal: its own un-rounded intermediate, quantised here with torch's
    e4m3 cast, times the dequantised down weights in float64.  A wrong group width, a wrong scale constant or a
    quantisation placed elsewhere on the path breaks the equality; the negative controls show the test sees them."""
    spec = synth.scaled(synth.SPECS["c5"], shape=synth.Shape(3, 2, 256, I, "fp8"), ops=((synth.PREFILL, 7),))
    sh = spec.shape
    Wt = synth.make_weights(spec, threads=2)
    op = synth.make_ops(spec)[0]
    W = oracle.Weights(sh.E, sh.k, sh.H, sh.I, Wt.w_gate_up, Wt.w_down, Wt.s_gate_up, Wt.s_down)
    row_token = np.repeat(np.arange(op.T, dtype=np.int32), sh.k)
    row_expert = op.ids.reshape(-1)
    _, A = oracle.ffn_rows(W, op.x, op.x_scale, row_token, row_expert, want_A=True)
    D_q = oracle.ffn_rows(W, op.x, op.x_scale, row_token, row_expert, round_A=oracle.ROUND_E4M3_1X128)
    w2 = _deq_blocks(Wt.w_down, Wt.s_down, 128, 128)               # [E, H, I] float64

    def down(Aq):
        return np.stack([(w2[int(e)] @ Aq[r]).numpy() for r, e in enumerate(row_expert)])

    scale = np.abs(D_q).max()
    expect = down(_quant_rows_torch(torch.from_numpy(A), 128))
    assert np.abs(D_q - expect).max() <= 1e-6 * scale
    # negative controls: one group per row, 64-wide groups, a scale of amax/240, and no rounding at all
    assert np.abs(D_q - down(_quant_rows_torch(torch.from_numpy(A), I))).max() > 1e-3 * scale
    assert np.abs(D_q - down(_quant_rows_torch(torch.from_numpy(A), 64))).max() > 1e-3 * scale
    assert np.abs(D_q - down(torch.from_numpy(A).to(torch.float64))).max() > 1e-3 * scale
    blk = torch.from_numpy(A).view(A.shape[0], I // 128, 128)
    amax = blk.abs().amax(dim=2, keepdim=True)
    wrong = ((blk * (240.0 / amax)).to(torch.float8_e4m3fn).to(torch.float32) * (amax / 240.0)).view(A.shape)
    assert np.abs(D_q - down(wrong.to(torch.float64))).max() > 1e-3 * scale


def test_bf16_rounding_switches_match_the_library_cast():
    """round_A / round_D = bf16 (the switches that localise a GPU mismatch to the stored intermediate or the
    stored expert output): A is cast to bf16 before the down projection, D after it -- each against torch's
    bfloat16 cast applied to the oracle's un-rounded values, the down projection redone in float64."""
    spec = synth.Spec("rb", synth.Shape(3, 2, 256, 384), ((synth.PREFILL, 6),), "uniform", None, 1.0, -1.0, 91)
    sh = spec.shape
    Wt = synth.make_weights(spec, threads=2)
    op = synth.make_ops(spec)[0]
    W = oracle.Weights(sh.E, sh.k, sh.H, sh.I, Wt.w_gate_up, Wt.w_down)
    row_token = np.repeat(np.arange(op.T, dtype=np.int32), sh.k)
    row_expert = op.ids.reshape(-1)
    D, A = oracle.ffn_rows(W, op.x, None, row_token, row_expert, want_A=True)
    w2 = Wt.w_down.to(torch.float64)
    A_b = torch.from_numpy(A).to(torch.bfloat16).to(torch.float64)
    expect_A = np.stack([(w2[int(e)] @ A_b[r]).numpy() for r, e in enumerate(row_expert)])
    got_A = oracle.ffn_rows(W, op.x, None, row_token, row_expert, round_A=oracle.ROUND_BF16)
    assert np.abs(got_A - expect_A).max() <= 1e-6 * np.abs(expect_A).max()
    assert np.abs(got_A - D).max() > 1e-4 * np.abs(D).max()         # the rounding is visible
    got_D = oracle.ffn_rows(W, op.x, None, row_token, row_expert, round_D=oracle.ROUND_BF16)
    assert np.array_equal(got_D, torch.from_numpy(D).to(torch.bfloat16).float().numpy())


def test_online_budget_closed_forms_and_brute_force():
    """Section 6.4: q' = min(Q_max, ceil_c(q x_moe / x_moe*)).  Closed forms, and exact rational arithmetic
    on a grid (a wrong rounding direction, a forgotten cap or a forgotten cluster multiple fails one)."""
    from fractions import Fraction
    ob = oracle.online_budget
    assert ob(32, 100, 100, 148, 1) == 32            # footprint as expected: the static budget
    assert ob(32, 200, 100, 148, 1) == 64            # twice the footprint: twice the budget
    assert ob(32, 1000, 100, 96, 1) == 96            # capped: Q_max preserves prefill progress
    assert ob(32, 0, 100, 148, 2) == 0               # nothing to run
    assert ob(3, 100, 100, 148, 2) == 4              # rounded UP to a cluster multiple
    assert ob(32, 101, 100, 148, 1) == 33            # ceil, not round
    for q in (0, 1, 7, 32, 64):
        for x in (0, 1, 5, 99, 100, 101, 250):
            for xs in (1, 3, 100, 128):
                for c in (1, 2, 4):
                    exact = Fraction(q * x, xs)
                    ceil = -((-exact.numerator) // exact.denominator)
                    ceil_c = -(-ceil // c) * c
                    assert ob(q, x, xs, 120, c) == min(120, ceil_c)
                    assert ob(q, x, xs, 120, c) % c == 0 or ob(q, x, xs, 120, c) == 120
