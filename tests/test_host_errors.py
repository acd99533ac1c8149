"""Host-side argument checks of the C ABI (no GPU work is launched by any of these calls) and the
capacity formula C = ceil(cf*T*k/E) of Sec. 2.3 / Algorithm 1 step 1 against the oracle's exact version."""
import ctypes as C

import pytest

from paper_2508_12801_b200 import binding as ms

OK, INVALID, INFEASIBLE, WORKSPACE, CUDA, NOT_CONVERGED, UNSUPPORTED = range(7)


def _status(**kw):
    base = dict(T=512, d_model=256, E=8, k=2, capacity_factor=1.0)
    base.update(kw)
    p = ms.make_params(**base)
    n = C.c_size_t(0)
    return ms._lib.maxscore_workspace_bytes(C.byref(p), C.byref(n)), n.value


def test_valid_params_give_a_workspace_size():
    s, n = _status()
    assert s == OK and n > 0
    s2, n2 = _status(T=65536, d_model=4096, E=128, k=8)
    assert s2 == OK and n2 > n


@pytest.mark.parametrize("kw,want", [
    (dict(T=0), INVALID), (dict(T=-5), INVALID), (dict(E=0), INVALID), (dict(k=0), INVALID), (dict(d_model=0), INVALID),
    (dict(t=0.0), INVALID), (dict(t=-1.0), INVALID), (dict(t=float("nan")), INVALID), (dict(t=float("inf")), INVALID),
    (dict(io_dtype=7), INVALID), (dict(score_mode=2), INVALID), (dict(w_gate_layout=3), INVALID),
    (dict(capacity_factor=0.0), INVALID), (dict(score_mode=1, quant_shift=15), INVALID), (dict(max_sweeps=-1), INVALID),
    (dict(softtopk_mode=3), INVALID), (dict(softtopk_mode=2), OK), (dict(softtopk_mode=1, rankscale_delta=2), INVALID),
    (dict(softtopk_mode=1, rankscale_beta=float("nan")), INVALID), (dict(softtopk_mode=1, rankscale_beta=1.0, rankscale_delta=1), OK),
    (dict(k=9, E=8), INFEASIBLE),                       # k > E
    (dict(capacity=100), INFEASIBLE),                   # 8 * 100 < 512 * 2
    (dict(capacity_factor=0.5), INFEASIBLE),            # C = 64: 8 * 64 < 1024
    (dict(T=4, E=8, k=2, capacity=8), OK),              # C >= T: every token can take any k experts
    (dict(E=129, k=2), UNSUPPORTED), (dict(E=64, k=9), UNSUPPORTED),
    (dict(d_model=252, io_dtype=ms.BF16), UNSUPPORTED), (dict(d_model=254, io_dtype=ms.F32), UNSUPPORTED),
    (dict(T=1 << 29, k=8, E=128, d_model=8), UNSUPPORTED),   # T * k must stay below 2^31
])
def test_bad_params_are_rejected_before_any_launch(kw, want):
    assert _status(**kw)[0] == want


def test_null_pointers():
    n = C.c_size_t(0)
    assert ms._lib.maxscore_workspace_bytes(None, C.byref(n)) == INVALID
    p = ms.make_params(512, 256, 8, 2)
    assert ms._lib.maxscore_workspace_bytes(C.byref(p), None) == INVALID
    assert ms._lib.maxscore_capacity(None) == -1


@pytest.mark.parametrize("T,E,k,num,den", [(512, 8, 2, 1, 1), (4096, 16, 2, 1, 1), (8192, 64, 8, 1, 1),
                                           (16384, 64, 8, 5, 4), (65536, 128, 8, 1, 1), (1000, 16, 2, 5, 4),
                                           (777, 64, 8, 1, 1), (33, 5, 5, 1, 1), (1001, 7, 3, 3, 2)])
def test_capacity_matches_the_exact_ceiling(orc, T, E, k, num, den):
    p = ms.make_params(T, 64, E, k, capacity_factor=num / den)
    assert ms.capacity(p) == orc.capacity(T, k, E, num / den)
