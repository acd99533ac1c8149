"""GPU parity, stage by stage: every CUDA stage is called through the C ABI and compared with the
CPU oracle on the same seeded inputs.  Downstream stages are fed the GPU's own upstream output, so
that a flipped near-tie upstream cannot pass for a downstream bug.

Tolerances.  SoftTopk sums positive terms, so it is held to 1e-5 relative elementwise.  Outputs that
are sums of signed products (gate, combine, the backward GEMMs) are held to
  fp32 outputs:  1e-5 * (the same sum over absolute values), and per row max|d| <= 1e-5 * max|ref|;
  bf16 outputs:  2^-8 * |ref| + 1e-5 * (the same sum over absolute values): one rounding of the result
                 plus fp32 accumulation; and per row max|d| <= 2e-2 * max|ref| as the outer bar."""
import numpy as np
import pytest
import torch

from gpu_util import (assert_rel, assert_rounded_sum_close, assert_row_rel, assert_sum_close, f64, float_keys, np32,
                      raw16)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ms():
    from paper_2508_12801_b200 import binding
    assert torch.cuda.is_available()
    return binding


@pytest.fixture(scope="module")
def synth():
    from paper_2508_12801_b200 import synth
    return synth


DEV = "cuda:0"


def _ctx(ms, T, d, E, k, cf=1.0, dtype="bf16", **kw):
    p = ms.make_params(T, d, E, k, cf, io_dtype=ms.BF16 if dtype == "bf16" else ms.F32, **kw)
    return ms.create(p, DEV)


def _tol(dtype):
    return 2e-2 if dtype == "bf16" else 1e-5


def _assert_out(got, ref, mag, dtype, what, rows=True):
    """An output in the I/O dtype: fp32 accumulation error, plus one rounding when the output is bf16."""
    if dtype == "bf16":
        assert_rounded_sum_close(got, ref, mag, 1e-5, what)
    else:
        assert_sum_close(got, ref, mag, 1e-5, what)
    if rows:
        assert_row_rel(got, ref, _tol(dtype), what + " (row-relative)")


# ------------------------------------------------------------------------------------------- gate
@pytest.mark.parametrize("T,d,E,dtype,layout,bias", [
    (512, 256, 8, "f32", 0, False), (300, 100, 12, "f32", 1, True),
    (512, 256, 8, "bf16", 0, False), (4096, 1024, 16, "bf16", 0, True),
    (1000, 2048, 64, "bf16", 1, False), (257, 4096, 128, "bf16", 0, True),
    (129, 72, 20, "bf16", 0, False),
])
def test_gate(ms, orc, synth, T, d, E, dtype, layout, bias):
    w = synth.Workload("g", T, d, E, 2, 1.0, dtype)
    H, W = synth.hidden(w, 1), synth.w_gate(w, 1)
    b = torch.linspace(-1, 1, E) if bias else None
    ctx = _ctx(ms, T, d, E, min(2, E), dtype=dtype, w_gate_layout=layout)
    Wd = (W if layout == 0 else W.t().contiguous()).to(DEV)
    L = torch.empty(T, E, dtype=torch.float32, device=DEV)
    ms.gate(ctx, H.to(DEV), Wd, b.to(DEV) if bias else None, L)
    torch.cuda.synchronize()
    ref = orc.gate(f64(H), f64(W), f64(b) if bias else None)
    mag = orc.gate(np.abs(f64(H)), np.abs(f64(W)), np.abs(f64(b)) if bias else None)
    assert_sum_close(np32(L), ref, mag, 1e-5, "gate")      # logits are fp32 in both I/O modes
    assert_row_rel(np32(L), ref, 1e-5, "gate (row-relative)")


# ------------------------------------------------------------------------------------------- SoftTopk
@pytest.mark.parametrize("T,E,k,t", [(512, 8, 2, 1.0), (512, 8, 2, 4.0), (1000, 16, 2, 1.0), (777, 64, 8, 1.0),
                                      (515, 128, 8, 0.25), (64, 20, 3, 2.0), (33, 5, 5, 1.0), (40, 128, 1, 1.0),
                                      # odd expert counts (the two lanes of a token get unequal shares), k = E (no tail),
                                      # several tiles with a ragged last one, every list width (k <= 2, <= 4, <= 8)
                                      (300, 77, 5, 1.0), (130, 8, 8, 0.5), (4133, 101, 4, 1.0), (257, 3, 1, 1.0), (1, 128, 8, 1.0)])
def test_softtopk_fwd_bwd(ms, orc, synth, T, E, k, t):
    L = synth.logits_like(T, E, seed=3)
    ctx = _ctx(ms, T, 64, E, k, cf=float(E), t=t)       # capacity irrelevant here
    Ld = L.to(DEV)
    A = torch.empty_like(Ld)
    ms.softtopk_fwd(ctx, Ld, A)
    ref = orc.softtopk_fwd(f64(L), k, t)
    assert_rel(np32(A), ref, 1e-5, "SoftTopk fwd")
    # backward with a sparse upstream gradient at k "assigned" experts per token
    g = torch.Generator().manual_seed(5)
    idx = torch.stack([torch.randperm(E, generator=g)[:k].sort().values for _ in range(T)]).to(torch.int32)
    dg = torch.randn(T, k, generator=g)
    dL = torch.empty_like(Ld)
    ms.softtopk_bwd(ctx, Ld, idx.to(DEV), dg.to(DEV), dL)
    G = np.zeros((T, E)); np.put_along_axis(G, idx.numpy().astype(np.int64), f64(dg), axis=1)
    refb = orc.softtopk_bwd(f64(L), G, k, t)
    got = np32(dL)
    rowmax = np.abs(refb).max(axis=1, keepdims=True)
    assert (np.abs(got - refb) <= 1e-5 * rowmax + 1e-9).all()


def _softtopk_against_oracle(ms, orc, L, k, t):
    T, E = L.shape
    ctx = _ctx(ms, T, 64, E, k, cf=float(E), t=t)
    Ld = L.to(DEV)
    A = torch.empty_like(Ld)
    ms.softtopk_fwd(ctx, Ld, A)
    assert_rel(np32(A), orc.softtopk_fwd(f64(L), k, t), 1e-5, "SoftTopk fwd")
    g = torch.Generator().manual_seed(5)
    idx = torch.stack([torch.randperm(E, generator=g)[:k].sort().values for _ in range(T)]).to(torch.int32)
    dg = torch.randn(T, k, generator=g)
    dL = torch.empty_like(Ld)
    ms.softtopk_bwd(ctx, Ld, idx.to(DEV), dg.to(DEV), dL)
    G = np.zeros((T, E)); np.put_along_axis(G, idx.numpy().astype(np.int64), f64(dg), axis=1)
    refb = orc.softtopk_bwd(f64(L), G, k, t)
    scale = np.abs(G).max(axis=1, keepdims=True) * (k / t)          # |J^T g| <= k/t * max|g| per row
    assert (np.abs(np32(dL) - refb) <= 1e-5 * scale + 1e-12).all()


@pytest.mark.parametrize("E,k,t", [(8, 2, 1.0), (64, 8, 1.0), (128, 8, 0.25), (20, 3, 2.0)])
def test_softtopk_tied_logits_take_the_lowest_index(ms, orc, synth, E, k, t):
    """Logits on a 0.25 grid tie often, and some rows are all equal: which entry a level masks is then decided
    by the lowest-expert-index rule, on both sides (Eq. 6's Topk is silent on ties)."""
    T = 384
    L = (synth.logits_like(T, E, seed=8) * 4).round() / 4
    L[5] = 0.5; L[6] = -3.0; L[7, : E // 2] = 1.0; L[7, E // 2:] = 1.0      # all-equal rows
    L[8] = 0.0; L[8, E - 1] = 2.0; L[8, 0] = 2.0                           # the maximum twice, far apart
    _softtopk_against_oracle(ms, orc, L, k, t)


@pytest.mark.parametrize("E,k,t", [(64, 8, 0.25), (128, 8, 0.25), (16, 4, 0.5)])
def test_softtopk_rows_whose_levels_fall_far_below_the_row_maximum(ms, orc, synth, E, k, t):
    """Widely spread logits (N(0,1) x 40 at a small temperature, and rows with one or two entries 100 t
    above the rest): a later level's maximum then lies more than 60 t below the first one's, which makes
    the kernel re-base its exponentials on that level's own maximum."""
    T = 256
    L = synth.logits_like(T, E, seed=9) * 40.0
    L[3] = synth.logits_like(1, E, seed=10)[0]; L[3, 2] += 100.0 * t
    L[4] = synth.logits_like(1, E, seed=11)[0]; L[4, 1] += 100.0 * t; L[4, E - 1] += 170.0 * t
    # the spread must really exceed the re-base threshold on most rows
    top = np.sort(f64(L), axis=1)[:, ::-1]
    assert ((top[:, 0] - top[:, k - 1]) > 60.0 * t).mean() > 0.5
    _softtopk_against_oracle(ms, orc, L, k, t)


@pytest.mark.parametrize("T,E,k,lam", [(512, 8, 2, 1e-2), (1000, 16, 2, 1e-2), (4099, 64, 8, 3e-3), (777, 128, 8, 1.0),
                                        (33, 5, 5, 0.5)])
def test_aux_loss_and_its_gradient_through_softtopk(ms, orc, synth, T, E, k, lam):
    """Eq. 9 on the GPU's own scores, and dlogits with its gradient folded into the SoftTopk backward."""
    lam = float(np.float32(lam))                         # the C ABI takes lambda as a float
    L = synth.logits_like(T, E, seed=7)
    ctx = _ctx(ms, T, 64, E, k, cf=float(E), t=1.0)
    Ld = L.to(DEV)
    A = torch.empty_like(Ld)
    ms.softtopk_fwd(ctx, Ld, A)
    g = torch.Generator().manual_seed(9)
    idx = torch.stack([torch.randperm(E, generator=g)[:k].sort().values for _ in range(T)]).to(torch.int32)
    load = torch.bincount(idx.flatten().long(), minlength=E).to(torch.int32)
    loss = torch.zeros(1, dtype=torch.float64, device=DEV)
    col = torch.empty(E, dtype=torch.float32, device=DEV)
    for _ in range(2):                                   # twice: the scratch must come back clean
        ms.aux_loss(ctx, A, load.to(DEV), lam, loss, col)
    torch.cuda.synchronize()
    An = np32(A).astype(np.float64)
    want = orc.aux_loss(An, idx.numpy(), lam)
    assert abs(loss.item() - want) <= 1e-12 * abs(want)          # double accumulation of the same fp32 scores
    gref = orc.aux_loss_grad(idx.numpy(), T, E, lam)
    np.testing.assert_allclose(np32(col), gref, rtol=1e-6, atol=0)
    # backward: dense per-expert term plus the sparse combine-weight gradients
    dg = torch.randn(T, k, generator=g)
    dL = torch.empty_like(Ld)
    ms.softtopk_bwd_aux(ctx, Ld, idx.to(DEV), dg.to(DEV), col, dL)
    G = np.tile(np32(col).astype(np.float64), (T, 1))
    G[np.arange(T)[:, None], idx.numpy().astype(np.int64)] += f64(dg)
    refb = orc.softtopk_bwd(f64(L), G, k, 1.0)
    got = np32(dL)
    scale = (np.abs(G).max(axis=1, keepdims=True))               # |J^T g| <= k/t * max|g| per row
    assert (np.abs(got - refb) <= 1e-5 * scale + 1e-12).all()


@pytest.mark.parametrize("T,E,k,t,beta,delta", [(512, 8, 2, 1.0, 0.0, 0), (1000, 16, 2, 0.5, 1.0, 1), (777, 64, 8, 1.0, 1.0, 1),
                                                 (515, 128, 8, 0.25, 0.0, 0), (33, 5, 5, 1.0, 0.0, 0), (64, 20, 3, 2.0, 1.0, 1)])
def test_softtopk_literal_readings_fwd_bwd(ms, orc, synth, T, E, k, t, beta, delta):
    """softtopk_mode 1: y = softmax(a) * (beta + t * min(rank - delta, k)) and its backward (ranks constant)."""
    L = synth.logits_like(T, E, seed=4)
    ctx = _ctx(ms, T, 64, E, k, cf=float(E), t=t, softtopk_mode=1, rankscale_beta=beta, rankscale_delta=delta)
    Ld = L.to(DEV)
    A = torch.empty_like(Ld)
    ms.softtopk_fwd(ctx, Ld, A)
    assert_rel(np32(A), orc.softtopk_rankscale_fwd(f64(L), k, t, beta, delta), 1e-5, "rank-scaled softmax fwd")
    g = torch.Generator().manual_seed(6)
    idx = torch.stack([torch.randperm(E, generator=g)[:k].sort().values for _ in range(T)]).to(torch.int32)
    dg = torch.randn(T, k, generator=g)
    col = torch.randn(E, generator=g) * 0.1
    dL = torch.empty_like(Ld)
    ms.softtopk_bwd_aux(ctx, Ld, idx.to(DEV), dg.to(DEV), col.to(DEV), dL)
    G = np.tile(f64(col), (T, 1))
    G[np.arange(T)[:, None], idx.numpy().astype(np.int64)] += f64(dg)
    ref = orc.softtopk_rankscale_bwd(f64(L), G, k, t, beta, delta)
    scale = np.abs(G).max(axis=1, keepdims=True) * (abs(beta) + t * k)      # |da| <= 2 * max|g s| per row
    assert (np.abs(np32(dL) - ref) <= 1e-5 * scale + 1e-12).all()
    ms.softtopk_bwd(ctx, Ld, idx.to(DEV), dg.to(DEV), dL)                    # without the dense term
    G2 = np.zeros((T, E)); np.put_along_axis(G2, idx.numpy().astype(np.int64), f64(dg), axis=1)
    ref2 = orc.softtopk_rankscale_bwd(f64(L), G2, k, t, beta, delta)
    assert (np.abs(np32(dL) - ref2) <= 1e-5 * scale + 1e-12).all()


def test_route_fwd_with_the_literal_reading(ms, orc, synth):
    """The solver does not care which reading produced the affinities: optimal for the scores it is given."""
    wl = synth.scaled(synth.WORKLOADS["k2e16"], T=2048, d_model=256)
    H, W = synth.hidden(wl), synth.w_gate(wl)
    ctx = ms.create(ms.make_params(wl.T, wl.d_model, wl.E, wl.k, 1.0, softtopk_mode=1, rankscale_beta=1.0,
                                   rankscale_delta=1), DEV)
    buf = ms.RouterBuffers(ctx)
    ms.route_fwd(ctx, H.to(DEV), W.to(DEV), None, *buf.args())
    torch.cuda.synchronize()
    assert ms.read_stats(buf.stats).status == 0
    L = np32(buf.logits); A = np32(buf.scores)
    assert_rel(A, orc.softtopk_rankscale_fwd(L.astype(np.float64), wl.k, 1.0, 1.0, 1), 1e-5, "scores")
    idx = buf.expert_idx.cpu().numpy()
    res, _ = orc.flow_certificate(float_keys(A), idx, ctx.capacity)
    assert res >= 1


# ------------------------------------------------------------------------------------------- assignment
def _run_assign(ms, M, T, E, k, cf, **kw):
    ctx = _ctx(ms, T, 64, E, k, cf=cf, **kw)
    idx = torch.empty(T, k, dtype=torch.int32, device=DEV)
    load = torch.empty(E, dtype=torch.int32, device=DEV)
    stats = ms.new_stats(DEV)
    Md = M.to(DEV)
    ms.assign(ctx, Md, idx, load, stats)
    torch.cuda.synchronize()
    return ctx, idx.cpu().numpy(), load.cpu().numpy(), ms.read_stats(stats)


def _describe(st):
    return (f"status={st.status} sweeps={st.sweeps} aug={st.augmentations} rounds={st.rounds} "
            f"cand={st.candidates} rerouted={st.rerouted}")


def _check_feasible(idx, load, T, E, k, C, st=None):
    msg = _describe(st) if st is not None else ""
    assert (idx >= 0).all() and (idx < E).all(), msg
    assert k == 1 or (np.diff(idx, axis=1) > 0).all(), msg
    np.testing.assert_array_equal(np.bincount(idx.ravel(), minlength=E), load, err_msg=msg)
    assert (load <= C).all() and load.sum() == T * k, f"{msg} load max {load.max()} C {C}"


@pytest.mark.parametrize("T,E,k,cf,skew", [(512, 8, 2, 1.0, False), (4096, 16, 2, 1.0, False),
                                            (1000, 16, 4, 1.0, False), (2048, 64, 8, 1.0, False),
                                            (2048, 64, 8, 1.25, True), (300, 8, 2, 1.5, True),
                                            (8192, 64, 8, 1.0, False), (129, 5, 5, 1.0, False),
                                            (257, 12, 1, 1.0, True),
                                            # a few units of spare room (T*k not a multiple of E): the sweeps hide them at first
                                            (4097, 16, 2, 1.0, False), (2051, 64, 8, 1.0, False), (8269, 128, 8, 1.0, False)])
def test_assign_float_scores(ms, orc, synth, T, E, k, cf, skew):
    wl = synth.Workload("a", T, 64, E, k, cf, "bf16", skew=skew)
    L = synth.logits_like(T, E, seed=7, bias=synth.expert_bias(wl, 7))
    A = torch.from_numpy(orc.softtopk_fwd(f64(L), k, 1.0).astype(np.float32))
    ctx, idx, load, st = _run_assign(ms, A, T, E, k, cf)
    C = ctx.capacity
    assert C == orc.capacity(T, k, E, cf)
    _check_feasible(idx, load, T, E, k, C, st)
    assert st.status == 0, _describe(st)
    # optimal for the keys the library documents ...
    keys = float_keys(A.numpy())
    res, prices = orc.flow_certificate(keys, idx, C)
    assert res >= 1, _describe(st)
    assert orc.dual_value(keys, prices, k, C) == orc.primal_value(keys, idx)
    # ... and within 1e-5 relative of the oracle's optimum of the float problem
    oidx, oload, _ = orc.flow_condensed(orc.keys_from_scores(f64(A)), k, C)
    best = orc.total_score(f64(A), oidx)
    got = orc.total_score(f64(A), idx)
    assert abs(got - best) <= 1e-5 * abs(best)
    assert abs(st.total_score - got) <= 1e-6 * abs(got)
    if cf == 1.0 and (T * k) % E == 0:
        assert (load == C).all()
    # rerouted = token-slots outside the token's own top-k
    topk = np.argsort(-keys, axis=1, kind="stable")[:, :k]
    inside = (idx[:, :, None] == topk[:, None, :]).any(2)
    assert st.rerouted == int((~inside).sum())


@pytest.mark.parametrize("T,E,k", [(4096, 64, 8), (16000, 64, 8), (6000, 100, 4)])
def test_assign_lopsided_router_with_every_expert_full(ms, orc, synth, T, E, k):
    """Zipf-biased router at capacity factor 1 with T*k a multiple of E: most pairs start on a few experts and every
    expert has to end up full, the unpopular ones included, which no token keeps among its cached experts.  The
    oracle's solver would take minutes here, so optimality is certified instead: the oracle's certificate of the
    GPU's assignment (complementary slackness on the documented keys) and exact duality."""
    wl = synth.Workload("a", T, 64, E, k, 1.0, "bf16", skew=True)
    L = synth.logits_like(T, E, seed=21, bias=synth.expert_bias(wl, 21))
    A = torch.from_numpy(orc.softtopk_fwd(f64(L), k, 1.0).astype(np.float32))
    ctx, idx, load, st = _run_assign(ms, A, T, E, k, 1.0)
    C = ctx.capacity
    assert E * C == T * k
    _check_feasible(idx, load, T, E, k, C, st)
    assert st.status == 0, _describe(st)
    assert (load == C).all()
    keys = float_keys(A.numpy())
    res, prices = orc.flow_certificate(keys, idx, C)
    assert res >= 1, _describe(st)
    assert orc.dual_value(keys, prices, k, C) == orc.primal_value(keys, idx)


@pytest.mark.parametrize("T,E,k,cf,skew,seed", [(512, 8, 2, 1.0, False, 0), (2048, 64, 8, 1.0, False, 0),
                                                 (2048, 64, 8, 1.25, True, 1), (8192, 64, 8, 1.0, False, 0),
                                                 (1000, 16, 3, 1.0, False, 2), (4097, 16, 2, 1.0, False, 0),
                                                 (2051, 64, 8, 1.0, False, 3)])
def test_assign_integer_keys_bit_exact(ms, orc, synth, T, E, k, cf, skew, seed):
    wl = synth.Workload("a", T, 64, E, k, cf, "bf16", skew=skew)
    L = synth.logits_like(T, E, seed=11, bias=synth.expert_bias(wl, 11))
    ctx, idx, load, st = _run_assign(ms, L, T, E, k, cf, score_mode=1, quant_shift=11, tiebreak_seed=seed)
    C = ctx.capacity
    _check_feasible(idx, load, T, E, k, C, st)
    keys, _ = orc.keys_from_logits(np32(L), k, 11, seed)
    oidx, oload, _ = orc.flow_condensed(keys, k, C)
    res, _ = orc.flow_certificate(keys, oidx, C)
    assert res == 2, "oracle optimum not unique for this seed"
    np.testing.assert_array_equal(idx, oidx, err_msg=_describe(st))
    np.testing.assert_array_equal(load, oload)
    assert st.status == 0


def test_assign_degenerate_inputs(ms, orc):
    # all scores equal: every assignment within capacity is optimal; must stay feasible and certified
    T, E, k = 256, 8, 2
    A = torch.full((T, E), 0.25)
    ctx, idx, load, st = _run_assign(ms, A, T, E, k, 1.0)
    _check_feasible(idx, load, T, E, k, ctx.capacity, st)
    assert orc.flow_certificate(float_keys(A.numpy()), idx, ctx.capacity)[0] >= 1
    # one hot expert for everybody
    A = torch.zeros(T, E); A[:, 3] = 1.0; A += torch.arange(E) * 1e-3
    ctx, idx, load, st = _run_assign(ms, A, T, E, k, 1.0)
    _check_feasible(idx, load, T, E, k, ctx.capacity, st)
    assert orc.flow_certificate(float_keys(A.numpy()), idx, ctx.capacity)[0] >= 1
    # loose capacity: plain per-token top-k
    g = torch.Generator().manual_seed(1)
    A = torch.rand(T, E, generator=g)
    ctx, idx, load, st = _run_assign(ms, A, T, E, k, float(E))
    want = np.sort(np.argsort(-float_keys(A.numpy()), axis=1, kind="stable")[:, :k], axis=1)
    np.testing.assert_array_equal(idx, want)
    assert st.augmentations == 0 and st.rerouted == 0


# ------------------------------------------------------------------------------------------- index / dispatch / combine
@pytest.mark.parametrize("T,d,E,k,cf,dtype", [(512, 256, 8, 2, 1.0, "f32"), (1000, 512, 16, 2, 1.25, "bf16"),
                                               (2048, 2048, 64, 8, 1.0, "bf16"), (333, 4096, 128, 8, 1.5, "bf16"),
                                               (100, 8200, 8, 2, 1.0, "bf16"), (65, 40, 4, 1, 2.0, "f32")])
def test_index_dispatch_combine_and_backward(ms, orc, synth, T, d, E, k, cf, dtype):
    wl = synth.Workload("m", T, d, E, k, cf, dtype)
    H = synth.hidden(wl, 2)
    L = synth.logits_like(T, E, seed=2)
    A = orc.softtopk_fwd(f64(L), k, 1.0)
    C = orc.capacity(T, k, E, cf)
    oidx, _, _ = orc.flow_condensed(orc.keys_from_scores(A), k, C)
    ctx = _ctx(ms, T, d, E, k, cf=cf, dtype=dtype)
    assert ctx.capacity == C
    idx = torch.from_numpy(oidx).to(DEV)
    slot_idx = torch.empty(T, k, dtype=torch.int32, device=DEV)
    slot_token = torch.empty(E, C, dtype=torch.int32, device=DEV)
    load = torch.empty(E, dtype=torch.int32, device=DEV)
    ms.index_build(ctx, idx, slot_idx, slot_token, load)
    o_slot, o_tok, o_load = orc.index_build(oidx, E, C)
    np.testing.assert_array_equal(slot_idx.cpu().numpy(), o_slot)
    np.testing.assert_array_equal(slot_token.cpu().numpy(), o_tok)
    np.testing.assert_array_equal(load.cpu().numpy(), o_load)
    # dispatch: bit-exact rows, zero padding
    Hd = H.to(DEV)
    xd = torch.full((E, C, d), 7.0, dtype=H.dtype, device=DEV)      # poison: padding must be overwritten
    ms.dispatch(ctx, Hd, idx, slot_idx, slot_token, xd)
    torch.cuda.synchronize()
    if dtype == "bf16":
        np.testing.assert_array_equal(raw16(xd), orc.dispatch(raw16(H), o_tok))
    else:
        np.testing.assert_array_equal(xd.cpu().numpy(), orc.dispatch(H.numpy(), o_tok))
    # combine on independent expert outputs
    g = torch.Generator().manual_seed(9)
    yexp = torch.randn(E, C, d, generator=g).to(H.dtype)
    gw = torch.from_numpy(orc.gate_weights(A, oidx).astype(np.float32))
    Y = torch.empty(T, d, dtype=H.dtype, device=DEV)
    yd, gwd = yexp.to(DEV), gw.to(DEV)
    ms.combine(ctx, yd, idx, slot_idx, gwd, Y)
    refY = orc.combine(f64(yexp), oidx, o_slot, f64(gw))
    magY = orc.combine(np.abs(f64(yexp)), oidx, o_slot, np.abs(f64(gw)))
    _assert_out(f64(Y), refY, magY, dtype, "combine")
    # unit weights + accumulate (dispatch backward into an existing gradient)
    base = torch.randn(T, d, generator=g).to(H.dtype)
    Y2 = base.clone().to(DEV)
    ms.combine(ctx, yd, idx, slot_idx, None, Y2, accumulate=1)
    ref2 = f64(base) + orc.combine(f64(yexp), oidx, o_slot, None)
    mag2 = np.abs(f64(base)) + orc.combine(np.abs(f64(yexp)), oidx, o_slot, None)
    _assert_out(f64(Y2), ref2, mag2, dtype, "combine accumulate")
    # combine backward
    dY = synth.upstream_grad(wl, 2)
    dyexp = torch.full((E, C, d), 3.0, dtype=H.dtype, device=DEV)
    dgw = torch.empty(T, k, dtype=torch.float32, device=DEV)
    ms.combine_bwd(ctx, dY.to(DEV), yd, idx, slot_idx, gwd, slot_token, dyexp, dgw)
    r_dyexp, r_dgw = orc.combine_bwd(f64(dY), f64(yexp), oidx, o_slot, f64(gw))
    _assert_out(f64(dyexp), r_dyexp, np.abs(r_dyexp), dtype, "dyexp", rows=False)     # padding rows exactly zero
    _, m_dgw = orc.combine_bwd(np.abs(f64(dY)), np.abs(f64(yexp)), oidx, o_slot, np.abs(f64(gw)))
    assert_sum_close(np32(dgw), r_dgw, m_dgw, 1e-5, "dgate_w")                         # fp32 dot of exact products


@pytest.mark.parametrize("T,d,E,dtype,layout", [(512, 256, 8, "f32", 0), (1000, 1024, 16, "bf16", 0),
                                                 (700, 2048, 64, "bf16", 1), (130, 72, 20, "f32", 1)])
def test_gate_bwd(ms, orc, synth, T, d, E, dtype, layout):
    wl = synth.Workload("b", T, d, E, 2, 1.0, dtype)
    H, W = synth.hidden(wl, 4), synth.w_gate(wl, 4)
    dL = synth.logits_like(T, E, seed=4) * 0.1
    ctx = _ctx(ms, T, d, E, 2, dtype=dtype, w_gate_layout=layout)
    Wd = (W if layout == 0 else W.t().contiguous()).to(DEV)
    dW = torch.empty(d, E, dtype=torch.float32, device=DEV)
    dH = torch.empty(T, d, dtype=H.dtype, device=DEV)
    ms.gate_bwd(ctx, H.to(DEV), Wd, dL.to(DEV), dW, dH)
    r_dW, r_dH = orc.gate_bwd(f64(H), f64(W), f64(dL))
    m_dW, m_dH = orc.gate_bwd(np.abs(f64(H)), np.abs(f64(W)), np.abs(f64(dL)))
    assert_sum_close(np32(dW), r_dW, m_dW, 1e-5, "dW")
    _assert_out(f64(dH), r_dH, m_dH, dtype, "dH")
    assert_row_rel(np32(dW), r_dW, 1e-5, "dW (row-relative)")


# ------------------------------------------------------------------------------------------- whole path
@pytest.mark.parametrize("name,T", [("tiny", None), ("k2e16", None), ("k8e64", 2048), ("skew", 2048)])
def test_route_fwd_end_to_end(ms, orc, synth, name, T):
    wl = synth.WORKLOADS[name]
    if T:
        wl = synth.scaled(wl, T=T)
    T, d, E, k = wl.T, wl.d_model, wl.E, wl.k
    H, W, b = synth.hidden(wl), synth.w_gate(wl), synth.expert_bias(wl)
    ctx = _ctx(ms, T, d, E, k, cf=wl.capacity_factor, dtype=wl.dtype)
    C = ctx.capacity
    buf = ms.RouterBuffers(ctx)
    Hd, Wd, bd = H.to(DEV), W.to(DEV), (b.to(DEV) if b is not None else None)
    ms.route_fwd(ctx, Hd, Wd, bd, *buf.args())
    torch.cuda.synchronize()
    st = ms.read_stats(buf.stats)
    assert st.status == 0 and st.capacity == C, _describe(st)
    L = np32(buf.logits); A = np32(buf.scores)
    refL = orc.gate(f64(H), f64(W), f64(b) if b is not None else None)
    magL = orc.gate(np.abs(f64(H)), np.abs(f64(W)), np.abs(f64(b)) if b is not None else None)
    assert_sum_close(L, refL, magL, 1e-5, "logits")
    assert_rel(A, orc.softtopk_fwd(L.astype(np.float64), k, 1.0), 1e-5, "scores from GPU logits")
    idx = buf.expert_idx.cpu().numpy(); load = buf.expert_load.cpu().numpy()
    _check_feasible(idx, load, T, E, k, C, st)
    keys = float_keys(A)
    assert orc.flow_certificate(keys, idx, C)[0] >= 1
    oidx, _, _ = orc.flow_condensed(orc.keys_from_scores(A.astype(np.float64)), k, C)
    best = orc.total_score(A.astype(np.float64), oidx)
    assert abs(orc.total_score(A.astype(np.float64), idx) - best) <= 1e-5 * abs(best)
    o_slot, o_tok, o_load = orc.index_build(idx, E, C)
    np.testing.assert_array_equal(buf.slot_idx.cpu().numpy(), o_slot)
    np.testing.assert_array_equal(buf.slot_token.cpu().numpy(), o_tok)
    np.testing.assert_array_equal(load, o_load)
    np.testing.assert_array_equal(np32(buf.gate_w), np.take_along_axis(A, idx.astype(np.int64), axis=1))


@pytest.mark.parametrize("name,T,bias", [("tiny", None, False), ("k2e16", 1000, False), ("skew", 2048, True),
                                         ("skew", 9000, True), ("stress", 8269, False)])
def test_route_dispatch_from_host_buffers(ms, orc, synth, name, T, bias):
    """The end-to-end entry point: batch in host memory in, indices and combine weights back in host memory,
    dispatched rows on the device.  Same kernels as route_fwd + dispatch, so the results are bit-identical to
    that path, and the dispatched rows are checked against the oracle.  The larger cases go up in eight row
    blocks with a ragged last one."""
    wl = synth.WORKLOADS[name]
    wl = synth.scaled(wl, T=T, d_model=min(wl.d_model, 512)) if T else wl
    T, d, E, k = wl.T, wl.d_model, wl.E, wl.k
    H, W = synth.hidden(wl), synth.w_gate(wl)
    b = synth.expert_bias(wl) if bias else None
    dt = H.dtype
    ctx = ms.create(ms.make_params(T, d, E, k, wl.capacity_factor, io_dtype=ms.BF16 if wl.dtype == "bf16" else ms.F32), DEV)
    C_ = ctx.capacity
    # device path
    buf = ms.RouterBuffers(ctx)
    Hd, Wd = H.to(DEV), W.to(DEV)
    bd = b.to(DEV) if b is not None else None
    ms.route_fwd(ctx, Hd, Wd, bd, *buf.args())
    xd = torch.empty(E, C_, d, dtype=dt, device=DEV)
    ms.dispatch(ctx, Hd, buf.expert_idx, buf.slot_idx, buf.slot_token, xd)
    torch.cuda.synchronize()
    want = [t.cpu().clone() for t in (buf.expert_idx, buf.slot_idx, buf.gate_w, buf.slot_token, buf.expert_load, xd)]
    # host path, fresh device staging buffers
    buf2 = ms.RouterBuffers(ctx)
    Hs, Ws = torch.empty_like(Hd), torch.empty_like(Wd)
    bs = torch.empty_like(bd) if bd is not None else None
    xd2 = torch.full((E, C_, d), 3.0, dtype=dt, device=DEV)
    dev = buf2.device_buffers(Hs, Ws, bs, xd2)
    idx_h = torch.empty(T, k, dtype=torch.int32).pin_memory()
    slot_h = torch.empty(T, k, dtype=torch.int32).pin_memory()
    gw_h = torch.empty(T, k, dtype=torch.float32).pin_memory()
    st_h = torch.zeros(40, dtype=torch.uint8).pin_memory()
    ms.route_dispatch_host(ctx, H.pin_memory(), W.pin_memory(), b.pin_memory() if b is not None else None, dev,
                           idx_h, slot_h, gw_h, st_h)
    torch.cuda.synchronize()
    assert ms.read_stats(st_h).status == 0
    assert torch.equal(idx_h, want[0]) and torch.equal(slot_h, want[1]) and torch.equal(gw_h, want[2])
    assert torch.equal(buf2.slot_token.cpu(), want[3]) and torch.equal(buf2.expert_load.cpu(), want[4])
    as_int = torch.int16 if dt == torch.bfloat16 else torch.int32
    assert torch.equal(xd2.cpu().view(as_int), want[5].view(as_int))
    o_slot, o_tok, _ = orc.index_build(idx_h.numpy(), E, C_)
    np.testing.assert_array_equal(slot_h.numpy(), o_slot)
    ref = orc.dispatch(H.view(as_int).numpy(), o_tok)
    np.testing.assert_array_equal(xd2.cpu().view(as_int).numpy(), ref)

@pytest.mark.parametrize("name", ["tiny", "k2e16"])
def test_route_bwd_whole_call_at_the_small_configs(ms, orc, synth, name):
    """maxscore_route_bwd as ONE call at the full shape of the two small workloads (fp32 I/O and bf16 I/O):
    forward on the GPU with identity experts (yexp = xdisp), upstream gradients N(0,1) over the combine
    output, then every output of the backward against the oracle's backward chain fed the GPU's own forward
    outputs (all rows)."""
    wl = synth.WORKLOADS[name]
    T, d, E, k = wl.T, wl.d_model, wl.E, wl.k
    H, W, dY = synth.hidden(wl), synth.w_gate(wl), synth.upstream_grad(wl)
    ctx = _ctx(ms, T, d, E, k, cf=wl.capacity_factor, dtype=wl.dtype)
    C = ctx.capacity
    buf = ms.RouterBuffers(ctx)
    Hd, Wd, dYd = H.to(DEV), W.to(DEV), dY.to(DEV)
    ms.route_fwd(ctx, Hd, Wd, None, *buf.args())
    xd = torch.empty(E, C, d, dtype=H.dtype, device=DEV)
    ms.dispatch(ctx, Hd, buf.expert_idx, buf.slot_idx, buf.slot_token, xd)
    dyexp = torch.full((E, C, d), 3.0, dtype=H.dtype, device=DEV)
    dgw = torch.empty(T, k, dtype=torch.float32, device=DEV)
    dL = torch.empty(T, E, dtype=torch.float32, device=DEV)
    dW = torch.empty(d, E, dtype=torch.float32, device=DEV)
    dH = torch.empty(T, d, dtype=H.dtype, device=DEV)
    ms.route_bwd(ctx, dYd, xd, Hd, Wd, buf.logits, buf.expert_idx, buf.slot_idx, buf.gate_w, buf.slot_token,
                 dyexp, dgw, dL, dW, dH)
    torch.cuda.synchronize()
    assert ms.read_stats(buf.stats).status == 0 and ms.check_internal(ctx) == 0
    idx = buf.expert_idx.cpu().numpy(); slot = buf.slot_idx.cpu().numpy()
    gw = np32(buf.gate_w).astype(np.float64); L = np32(buf.logits).astype(np.float64)
    yexp = f64(xd)
    r_dyexp, r_dgw = orc.combine_bwd(f64(dY), yexp, idx, slot, gw)
    _, m_dgw = orc.combine_bwd(np.abs(f64(dY)), np.abs(yexp), idx, slot, np.abs(gw))
    _assert_out(f64(dyexp), r_dyexp, np.abs(r_dyexp), wl.dtype, "dyexp", rows=False)
    assert_sum_close(np32(dgw), r_dgw, m_dgw, 1e-5, "dgate_w")
    # SoftTopk backward on the GPU's own dgate_w, gate backward on the GPU's own dlogits
    G = np.zeros((T, E)); np.put_along_axis(G, idx.astype(np.int64), np32(dgw).astype(np.float64), axis=1)
    r_dL = orc.softtopk_bwd(L, G, k, wl.temperature)
    scale = np.abs(G).max(axis=1, keepdims=True) * (k / wl.temperature)
    assert (np.abs(np32(dL) - r_dL) <= 1e-5 * scale + 1e-12).all()
    dLf = np32(dL).astype(np.float64)
    r_dW, r_dH = orc.gate_bwd(f64(H), f64(W), dLf)
    m_dW, m_dH = orc.gate_bwd(np.abs(f64(H)), np.abs(f64(W)), np.abs(dLf))
    assert_sum_close(np32(dW), r_dW, m_dW, 1e-5, "dW")
    assert_row_rel(np32(dW), r_dW, 1e-5, "dW (row-relative)")
    _assert_out(f64(dH), r_dH, m_dH, wl.dtype, "dH")


@pytest.mark.parametrize("T,E,k", [(512, 8, 2), (1000, 16, 2), (777, 64, 8), (515, 128, 8), (33, 5, 3), (64, 20, 1)])
def test_itertopk_of_table_2_fwd_bwd(ms, orc, synth, T, E, k):
    """softtopk_mode 2: IterTopk as Table 2 prints it, forward and backward, against the oracle."""
    L = synth.logits_like(T, E, seed=12)
    ctx = _ctx(ms, T, 64, E, k, cf=float(E), softtopk_mode=2)
    Ld = L.to(DEV)
    A = torch.empty_like(Ld)
    ms.softtopk_fwd(ctx, Ld, A)
    ref = orc.itertopk_fwd(f64(L), k)
    assert_row_rel(np32(A), ref, 1e-5, "IterTopk fwd")          # later levels subtract: held to the row maximum
    assert np.abs(np32(A).sum(axis=1) - k).max() <= 1e-4
    g = torch.Generator().manual_seed(13)
    idx = torch.stack([torch.randperm(E, generator=g)[:k].sort().values for _ in range(T)]).to(torch.int32)
    dg = torch.randn(T, k, generator=g)
    col = torch.randn(E, generator=g) * 0.1
    dL = torch.empty_like(Ld)
    ms.softtopk_bwd_aux(ctx, Ld, idx.to(DEV), dg.to(DEV), col.to(DEV), dL)
    G = np.tile(f64(col), (T, 1))
    G[np.arange(T)[:, None], idx.numpy().astype(np.int64)] += f64(dg)
    refb = orc.itertopk_bwd(f64(L), G, k)
    scale = np.abs(G).max(axis=1, keepdims=True) * k
    assert (np.abs(np32(dL) - refb) <= 2e-5 * scale + 1e-12).all()


@pytest.mark.parametrize("T,E,k,cf,skew", [(512, 8, 2, 1.0, False), (4096, 16, 2, 1.0, False), (1000, 16, 4, 1.0, False),
                                            (2048, 64, 8, 1.0, False), (2048, 64, 8, 1.25, True), (300, 8, 2, 1.5, True),
                                            (8192, 64, 8, 1.0, False), (129, 5, 5, 1.0, False), (3000, 128, 8, 1.0, True),
                                            (16384, 64, 8, 1.0, True), (20000, 32, 4, 1.0, True), (40000, 128, 8, 1.0, False)])
def test_iterative_rerouting_bit_exact(ms, orc, synth, T, E, k, cf, skew):
    """maxscore_assign_iterative against the oracle's top-k-with-capacity + greedy rerouting: with both serving
    orders fixed the result is unique, so everything is compared bit for bit.  Also: how far the greedy result
    is from the exact flow's optimum on the same scores."""
    wl = synth.Workload("a", T, 64, E, k, cf, "bf16", skew=skew)
    L = synth.logits_like(T, E, seed=14, bias=synth.expert_bias(wl, 14))
    A = torch.from_numpy(orc.softtopk_fwd(f64(L), k, 1.0).astype(np.float32))
    ctx = _ctx(ms, T, 64, E, k, cf=cf)
    C = ctx.capacity
    idx = torch.empty(T, k, dtype=torch.int32, device=DEV)
    load = torch.empty(E, dtype=torch.int32, device=DEV)
    counts = torch.full((2,), -1, dtype=torch.int32, device=DEV)
    for _ in range(2):                                    # twice: the workspace must come back usable
        ms.assign_iterative(ctx, A.to(DEV), idx, load, counts)
    torch.cuda.synchronize()
    oidx, oload, ond, one = orc.iterative_reroute(f64(A), k, C)
    np.testing.assert_array_equal(idx.cpu().numpy(), oidx)
    np.testing.assert_array_equal(load.cpu().numpy(), oload)
    assert counts.cpu().tolist() == [ond, one]
    assert (oload <= C).all()
    # the slots of the greedy assignment go through the same index build (empty slots are skipped)
    slot_idx = torch.empty(T, k, dtype=torch.int32, device=DEV)
    slot_token = torch.empty(E, C, dtype=torch.int32, device=DEV)
    load2 = torch.empty(E, dtype=torch.int32, device=DEV)
    ms.index_build(ctx, idx, slot_idx, slot_token, load2)
    np.testing.assert_array_equal(load2.cpu().numpy(), oload)
    # greedy is feasible, never better than the flow's optimum (checked where the exact solver on the CPU takes seconds)
    if one == 0 and T <= 8192:
        fidx, _, _ = orc.flow_condensed(orc.keys_from_scores(f64(A)), k, C)
        assert orc.total_score(f64(A), oidx) <= orc.total_score(f64(A), fidx) * (1 + 1e-12)


@pytest.mark.parametrize("T,E,cf,skew,eps,iters", [(512, 8, 1.0, False, 0.05, 8), (4096, 16, 1.0, False, 0.05, 16),
                                                   (1000, 16, 1.25, True, 0.1, 10), (3000, 64, 1.0, False, 0.02, 12),
                                                   (2048, 128, 1.0, True, 0.05, 6), (257, 5, 2.0, False, 0.05, 0)])
def test_algorithm_1_top1_then_sinkhorn(ms, orc, synth, T, E, cf, skew, eps, iters):
    """maxscore_assign_top2_sinkhorn against the oracle's Algorithm 1: the plan within 1e-9, every discrete output
    (the two experts per token, loads, drop counts) bit for bit.  Also the approximate-versus-exact comparison the
    paper motivates Algorithm 1 with: total score against the exact flow's, and the mean load ratio."""
    k = 2
    wl = synth.Workload("a", T, 64, E, k, cf, "bf16", skew=skew)
    L = synth.logits_like(T, E, seed=15, bias=synth.expert_bias(wl, 15))
    A = torch.from_numpy(orc.softtopk_fwd(f64(L), k, 1.0).astype(np.float32))
    eps = float(np.float32(eps))                          # the C ABI takes the regulariser as a float
    ctx = _ctx(ms, T, 64, E, k, cf=cf)
    C = ctx.capacity
    idx = torch.empty(T, k, dtype=torch.int32, device=DEV)
    load = torch.empty(E, dtype=torch.int32, device=DEV)
    plan = torch.empty(T, E, dtype=torch.float64, device=DEV)
    counts = torch.full((2,), -1, dtype=torch.int32, device=DEV)
    for _ in range(2):
        ms.assign_top2_sinkhorn(ctx, A.to(DEV), eps, iters, idx, load, plan, counts)
    torch.cuda.synchronize()
    first, second, resid, over, dropped, oplan = orc.alg1_top1_sinkhorn(f64(A), C, eps, iters, want_plan=True)
    got_plan = plan.cpu().numpy()
    assert np.abs(got_plan - oplan).max() <= 1e-9
    # where the oracle's own arg-max is decided by less than the plan tolerance, either choice is right
    srt = np.sort(oplan, axis=1)
    clear = (srt[:, -1] - srt[:, -2]) > 1e-8
    want = np.stack([np.where((second >= 0) & (second < first), second, first),
                     np.where((second >= 0) & (second < first), first, second)], axis=1).astype(np.int32)
    got = idx.cpu().numpy()
    assert clear.mean() > 0.99
    if clear.all():
        np.testing.assert_array_equal(got, want)
        oload = np.bincount(first, minlength=E) + np.bincount(second[second >= 0], minlength=E)
        np.testing.assert_array_equal(load.cpu().numpy(), oload)
        assert counts.cpu().tolist() == [over, dropped]
    else:
        np.testing.assert_array_equal(got[clear][:, 0] >= 0, want[clear][:, 0] >= 0)
    # approximate versus exact: the flow's optimum bounds Algorithm 1's score from above when nothing was dropped
    gl = load.cpu().numpy()
    if dropped == 0 and over == 0:
        fidx, _, _ = orc.flow_condensed(orc.keys_from_scores(f64(A)), k, C)
        assert orc.total_score(f64(A), got) <= orc.total_score(f64(A), fidx) * (1 + 1e-12)
    assert gl.sum() == 2 * T - dropped
