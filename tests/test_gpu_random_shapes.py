"""Randomly drawn shapes (seeded): expert counts that are not multiples of 32, any k up to 8, token counts that
leave a few units of spare room or none, loose and tight capacity, even and Zipf-skewed routers, logits on a coarse
grid (ties).  For each shape the two assignment entry points are compared with the oracle: iterative rerouting bit
for bit (Sec. 2.3; both serving orders fixed), the exact flow (Eq. 7-8) by feasibility, its status and the total
routed score against the oracle's optimum."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ms():
    from paper_2508_12801_b200 import binding
    assert torch.cuda.is_available()
    return binding


@pytest.fixture(scope="module")
def synth():
    from paper_2508_12801_b200 import synth
    return synth


def _cases(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < n:
        E = int(rng.integers(2, 129)); k = int(rng.integers(1, min(E, 8) + 1)); T = int(rng.integers(1, 2500))
        cf = float(rng.choice([1.0, 1.0, 1.05, 1.25, 2.0])); skew = bool(rng.integers(0, 2)); grid = bool(rng.integers(0, 4) == 0)
        out.append((T, E, k, cf, skew, grid, len(out)))
    return out


@pytest.mark.parametrize("T,E,k,cf,skew,grid,seed", _cases(32, 20240))
def test_assignments_on_random_shapes(ms, orc, synth, T, E, k, cf, skew, grid, seed):
    wl = synth.Workload("a", T, 64, E, k, cf, "bf16", skew=skew)
    L = synth.logits_like(T, E, seed=seed, bias=synth.expert_bias(wl, seed))
    if grid:
        L = torch.round(L * 2) / 2
    A64 = orc.softtopk_fwd(L.double().numpy(), k, 1.0).astype(np.float32).astype(np.float64)
    A = torch.from_numpy(A64.astype(np.float32)).to(DEV)
    ctx = ms.create(ms.make_params(T, 64, E, k, cf), DEV)
    C = ctx.capacity
    idx = torch.empty(T, k, dtype=torch.int32, device=DEV)
    load = torch.empty(E, dtype=torch.int32, device=DEV)
    counts = torch.full((2,), -1, dtype=torch.int32, device=DEV)
    ms.assign_iterative(ctx, A, idx, load, counts)
    torch.cuda.synchronize()
    oidx, oload, ond, one = orc.iterative_reroute(A64, k, C)
    np.testing.assert_array_equal(idx.cpu().numpy(), oidx)
    np.testing.assert_array_equal(load.cpu().numpy(), oload)
    assert counts.cpu().tolist() == [ond, one]

    stats = ms.new_stats(DEV)
    ms.assign(ctx, A, idx, load, stats)
    torch.cuda.synchronize()
    st = ms.read_stats(stats)
    got_idx = idx.cpu().numpy()
    assert st.status == 0, f"status {st.status} sweeps {st.sweeps} augmentations {st.augmentations} rounds {st.rounds}"
    assert ((got_idx >= 0) & (got_idx < E)).all() and (np.diff(np.sort(got_idx, axis=1), axis=1) > 0).all()
    l2 = np.bincount(got_idx.ravel(), minlength=E)
    np.testing.assert_array_equal(l2, load.cpu().numpy())
    assert l2.max() <= C
    fidx, _, _ = orc.flow_condensed(orc.keys_from_scores(A64), k, C)
    best, got = orc.total_score(A64, fidx), orc.total_score(A64, got_idx)
    assert abs(got - best) <= 1e-5 * abs(best) + 1e-12
