"""Error behaviour of the C ABI on a GPU: host-detectable errors come back as a status before any
launch; device-detected conditions come back as bits of stats.status, and the context stays usable."""
import ctypes as C

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
INVALID, WORKSPACE = 1, 3
STAT_NOT_CONVERGED, STAT_NON_FINITE, STAT_INTERNAL = 1, 2, 4


@pytest.fixture(scope="module")
def ms():
    from paper_2508_12801_b200 import binding
    assert torch.cuda.is_available()
    return binding


@pytest.fixture(scope="module")
def synth():
    from paper_2508_12801_b200 import synth
    return synth


def _solver_buffers(ms, T, E, k):
    idx = torch.empty(T, k, dtype=torch.int32, device=DEV)
    load = torch.empty(E, dtype=torch.int32, device=DEV)
    return idx, load, ms.new_stats(DEV)


def test_short_or_misaligned_workspace_is_rejected(ms):
    p = ms.make_params(512, 256, 8, 2)
    n = ms.workspace_bytes(p)
    ws = torch.empty(n + 512, dtype=torch.uint8, device=DEV)
    base = (ws.data_ptr() + 255) // 256 * 256
    h = C.c_void_p()
    assert ms._lib.maxscore_create(C.byref(h), C.byref(p), C.c_void_p(base), C.c_size_t(n - 1)) == WORKSPACE
    assert ms._lib.maxscore_create(C.byref(h), C.byref(p), C.c_void_p(base + 8), C.c_size_t(n)) == INVALID
    assert ms._lib.maxscore_create(C.byref(h), C.byref(p), None, C.c_size_t(n)) == INVALID
    assert ms._lib.maxscore_create(None, C.byref(p), C.c_void_p(base), C.c_size_t(n)) == INVALID
    assert not h.value


def test_null_and_misaligned_buffers_return_a_status(ms, synth):
    T, d, E, k = 512, 256, 8, 2
    ctx = ms.create(ms.make_params(T, d, E, k, io_dtype=ms.F32), DEV)
    M = torch.rand(T, E, device=DEV)
    idx, load, st = _solver_buffers(ms, T, E, k)
    with pytest.raises(ms.MaxScoreError) as e:
        ms.assign(ctx, None, idx, load, st)
    assert e.value.status == INVALID
    odd = torch.rand(T * E + 1, device=DEV)[1:].view(T, E)          # 4-byte aligned only
    with pytest.raises(ms.MaxScoreError) as e:
        ms.assign(ctx, odd, idx, load, st)
    assert e.value.status == INVALID
    ms.assign(ctx, M, idx, load, st)                                # the context is still good
    torch.cuda.synchronize()
    assert ms.read_stats(st).status == 0


def test_non_finite_scores_set_a_status_bit_and_nothing_faults(ms):
    T, E, k = 1024, 16, 2
    ctx = ms.create(ms.make_params(T, 64, E, k), DEV)
    g = torch.Generator().manual_seed(0)
    M = torch.rand(T, E, generator=g)
    M[3, 5] = float("nan"); M[700, 0] = float("inf"); M[701, 15] = -float("inf")
    idx, load, st = _solver_buffers(ms, T, E, k)
    ms.assign(ctx, M.to(DEV), idx, load, st)
    torch.cuda.synchronize()
    s = ms.read_stats(st)
    assert s.status & STAT_NON_FINITE
    ii = idx.cpu().numpy()
    assert ii.min() >= 0 and ii.max() < E and (np.diff(ii, axis=1) > 0).all()     # still k distinct experts each
    assert load.sum().item() == T * k
    # a clean matrix afterwards: the bit is gone
    ms.assign(ctx, torch.rand(T, E, generator=g).to(DEV), idx, load, st)
    torch.cuda.synchronize()
    assert ms.read_stats(st).status == 0


def test_exhausted_budget_reports_not_converged_and_downstream_stays_in_bounds(ms, orc, synth):
    """max_sweeps = 1 leaves no room for the exact phase: the result is top-k under the first prices.
    It must say so, keep k distinct experts per token, and index/dispatch/combine must skip what does
    not fit (slot >= C) instead of writing out of bounds."""
    T, d, E, k = 2048, 256, 16, 2
    wl = synth.scaled(synth.WORKLOADS["k2e16"], T=T, d_model=d)
    H, W = synth.hidden(wl), synth.w_gate(wl)
    # a strong per-expert bias: plain top-k overloads the favoured experts several-fold, so one price sweep and
    # no augmentation cannot possibly balance the load
    bias = torch.linspace(3.0, -3.0, E)
    ctx = ms.create(ms.make_params(T, d, E, k, 1.0, max_sweeps=1), DEV)
    C_ = ctx.capacity
    buf = ms.RouterBuffers(ctx)
    Hd = H.to(DEV)
    ms.route_fwd(ctx, Hd, W.to(DEV), bias.to(DEV), *buf.args())
    torch.cuda.synchronize()
    s = ms.read_stats(buf.stats)
    idx = buf.expert_idx.cpu().numpy(); load = buf.expert_load.cpu().numpy()
    assert idx.min() >= 0 and idx.max() < E and (np.diff(idx, axis=1) > 0).all()
    np.testing.assert_array_equal(np.bincount(idx.ravel(), minlength=E), load)
    assert load.sum() == T * k
    assert (load > C_).any(), "the input was built to stay out of balance"
    assert s.status & STAT_NOT_CONVERGED
    guard = torch.full((E * C_ + 8, d), 7.0, dtype=torch.bfloat16, device=DEV)       # canary rows behind the buffer
    xd = guard[:E * C_].view(E, C_, d)
    ms.dispatch(ctx, Hd, buf.expert_idx, buf.slot_idx, buf.slot_token, xd)
    Y = torch.empty(T, d, dtype=torch.bfloat16, device=DEV)
    ms.combine(ctx, xd, buf.expert_idx, buf.slot_idx, buf.gate_w, Y)
    torch.cuda.synchronize()
    assert (guard[E * C_:] == 7.0).all()
    # surplus pairs contribute zero and their row is not even read: an Inf in the first row of the buffer
    # reaches only the token that really sits there
    yexp = xd.clone(); yexp[0, 0, :] = float("inf")
    Y2 = torch.empty_like(Y)
    ms.combine(ctx, yexp, buf.expert_idx, buf.slot_idx, buf.gate_w, Y2)
    torch.cuda.synchronize()
    owner = int(buf.slot_token[0, 0].item())
    not_finite = np.where(~torch.isfinite(Y2.float()).all(dim=1).cpu().numpy())[0]
    assert set(not_finite.tolist()) <= {owner}
    tok = buf.slot_token.cpu().numpy()
    assert tok.shape == (E, C_) and tok.max() < T
    filled = tok >= 0
    assert filled.sum() == np.minimum(load, C_).sum()
    Hraw = H.view(torch.int16).numpy()
    got = xd.cpu().view(torch.int16).numpy()
    np.testing.assert_array_equal(got[filled], Hraw[tok[filled]])
    assert (got[~filled] == 0).all()


def test_internal_error_flag_reaches_the_caller(ms, synth):
    """The flag a bounded wait raises when it runs out is set here from the HOST (nothing waits or faults):
    route_fwd / assign must report it as MAXSCORE_STAT_INTERNAL and clear it; after a call that writes no stats
    maxscore_check_internal must return it once."""
    T, d, E, k = 1024, 256, 16, 2
    wl = synth.scaled(synth.WORKLOADS["k2e16"], T=T, d_model=d)
    H, W = synth.hidden(wl), synth.w_gate(wl)
    ctx = ms.create(ms.make_params(T, d, E, k, 1.0), DEV)
    buf = ms.RouterBuffers(ctx)
    Hd, Wd = H.to(DEV), W.to(DEV)
    ms.route_fwd(ctx, Hd, Wd, None, *buf.args())
    torch.cuda.synchronize()
    assert ms.read_stats(buf.stats).status == 0 and ms.check_internal(ctx) == 0
    ms.test_raise_internal(ctx)                           # as if a wait in a gate kernel had given up
    ms.route_fwd(ctx, Hd, Wd, None, *buf.args())
    torch.cuda.synchronize()
    assert ms.read_stats(buf.stats).status & STAT_INTERNAL
    ms.route_fwd(ctx, Hd, Wd, None, *buf.args())          # reported once, then gone
    torch.cuda.synchronize()
    assert ms.read_stats(buf.stats).status == 0
    # backward calls write no stats: the query returns the flag and clears it
    dL = torch.zeros(T, E, dtype=torch.float32, device=DEV)
    dW = torch.empty(d, E, dtype=torch.float32, device=DEV)
    dH = torch.empty(T, d, dtype=torch.bfloat16, device=DEV)
    ms.gate_bwd(ctx, Hd, Wd, dL, dW, dH)
    assert ms.check_internal(ctx) == 0
    ms.test_raise_internal(ctx)
    ms.gate_bwd(ctx, Hd, Wd, dL, dW, dH)
    assert ms.check_internal(ctx) != 0 and ms.check_internal(ctx) == 0
