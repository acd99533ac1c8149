"""Pins for the oracle's gate and SoftTopk (Eq. 2, Eq. 6) against things other than itself."""
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.special

HERE = os.path.dirname(os.path.abspath(__file__))


def test_gate_matches_library_matmul(orc):
    rng = np.random.default_rng(0)
    H = rng.standard_normal((37, 53))
    W = rng.standard_normal((53, 7))
    b = rng.standard_normal(7)
    np.testing.assert_allclose(orc.gate(H, W), H @ W, rtol=0, atol=1e-12)
    np.testing.assert_allclose(orc.gate(H, W, b), H @ W + b, rtol=0, atol=1e-12)
    # a transposed or mis-strided W would fail this asymmetric shape
    e3 = np.zeros((1, 53)); e3[0, 3] = 1.0
    np.testing.assert_array_equal(orc.gate(e3, W)[0], W[3])


def test_capacity_formula(orc):
    # C = cf*k*n/e for the five workloads (Sec. 2.3), all integers without rounding
    assert orc.capacity(512, 2, 8, 1.0) == 128
    assert orc.capacity(4096, 2, 16, 1.0) == 512
    assert orc.capacity(8192, 8, 64, 1.0) == 1024
    assert orc.capacity(16384, 8, 64, 1.25) == 2560
    assert orc.capacity(65536, 8, 128, 1.0) == 4096
    assert orc.capacity(7, 2, 4, 1.0) == 4          # ceil(3.5)
    assert orc.feasible(7, 2, 4, 4) and not orc.feasible(7, 2, 4, 3)
    assert not orc.feasible(4, 5, 4, 100)            # k > E
    assert not orc.feasible(4, 2, 2, 100) or orc.feasible(4, 2, 2, 4)
    assert orc.feasible(4, 2, 2, 100)                # C above T is clipped to T, still enough


def test_hand_case_from_section_3_1(orc):
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "softtopk_hand_case.txt"))
            if l.strip() and not l.startswith("#")]
    p = np.array([float(r[0]) for r in rows])
    want = np.array([float(r[1]) for r in rows])
    got = orc.softtopk_fwd(np.log(p)[None, :], k=2, t=1.0)[0]
    np.testing.assert_allclose(got, want, rtol=1e-12)


def _closed_form(a, k, t):
    """Sorted closed form: y_i = z_i * sum_{j < min(rank_i, k)} 1/Z_j, rank from 1,
    Z_j = sum of z over all but the j largest (independent restatement)."""
    a = np.asarray(a, dtype=np.float64)
    order = np.argsort(-a, kind="stable")
    z = np.exp((a - a.max()) / t)
    zs = z[order]
    tail = np.cumsum(zs[::-1])[::-1]           # tail[j] = sum_{r >= j} zs[r]
    y = np.empty_like(a)
    for r, i in enumerate(order):              # r = rank - 1
        y[i] = z[i] * sum(1.0 / tail[j] for j in range(min(r + 1, k)))
    return y


@pytest.mark.parametrize("E,k,t", [(8, 2, 1.0), (16, 2, 4.0), (64, 8, 1.0), (128, 8, 0.25), (5, 5, 2.0)])
def test_properties_and_closed_form(orc, E, k, t):
    rng = np.random.default_rng(E * 100 + k)
    L = rng.standard_normal((50, E)) * 2.0
    A = orc.softtopk_fwd(L, k, t)
    # every level is a probability vector, so the result sums to k
    np.testing.assert_allclose(A.sum(1), k, rtol=1e-12)
    assert (A > 0).all() and (A <= k + 1e-12).all()
    # closed form
    for r in range(10):
        np.testing.assert_allclose(A[r], _closed_form(L[r], k, t), rtol=1e-11)
    # shift invariance
    np.testing.assert_allclose(orc.softtopk_fwd(L + 3.25, k, t), A, rtol=1e-11)
    # permutation equivariance
    perm = rng.permutation(E)
    np.testing.assert_allclose(orc.softtopk_fwd(L[:, perm], k, t), A[:, perm], rtol=1e-12)
    # the largest entry is masked after level 1: its value is the plain softmax probability
    sm = scipy.special.softmax(L / t, axis=1)
    top = L.argmax(1)
    np.testing.assert_allclose(A[np.arange(50), top], sm[np.arange(50), top], rtol=1e-11)


def test_k1_is_softmax_with_temperature(orc):
    rng = np.random.default_rng(1)
    L = rng.standard_normal((20, 16))
    for t in (4.0, 1.0, 0.25):
        np.testing.assert_allclose(orc.softtopk_fwd(L, 1, t), scipy.special.softmax(L / t, axis=1), rtol=1e-12)


def test_small_t_tends_to_argtopk(orc):
    # Eq. 3: one-hot top-k indicator is the t -> 0 limit
    rng = np.random.default_rng(2)
    L = np.stack([rng.permutation(16) * 0.1 - 0.8 for _ in range(20)])   # gaps of 0.1 >> t
    A = orc.softtopk_fwd(L, 4, 1e-3)
    want = np.zeros_like(L)
    np.put_along_axis(want, np.argsort(-L, axis=1)[:, :4], 1.0, axis=1)
    np.testing.assert_allclose(A, want, atol=1e-9)


def test_equal_logits_closed_form_and_tie_rule(orc):
    # all logits equal, E=4, k=2: the lowest index is masked after level 1
    A = orc.softtopk_fwd(np.zeros((1, 4)), 2, 1.0)[0]
    want = [Fraction(1, 4), Fraction(1, 4) + Fraction(1, 3), Fraction(7, 12), Fraction(7, 12)]
    np.testing.assert_allclose(A, [float(x) for x in want], rtol=1e-14)
    # E=6, k=3: index 0 gets 1/6, index 1 gets 1/6+1/5, the rest 1/6+1/5+1/4
    A = orc.softtopk_fwd(np.full((1, 6), -2.5), 3, 0.7)[0]
    f = [Fraction(1, 6), Fraction(1, 6) + Fraction(1, 5)] + [Fraction(1, 6) + Fraction(1, 5) + Fraction(1, 4)] * 4
    np.testing.assert_allclose(A, [float(x) for x in f], rtol=1e-14)


def test_bad_arguments(orc):
    with pytest.raises(ValueError):
        orc.softtopk_fwd(np.zeros((1, 4)), 5, 1.0)
    with pytest.raises(ValueError):
        orc.softtopk_fwd(np.zeros((1, 4)), 2, 0.0)


# ---------------------------------------------------------------- backward
@pytest.mark.parametrize("E,k,t", [(8, 2, 1.0), (16, 4, 4.0), (12, 3, 0.5)])
def test_bwd_finite_differences(orc, E, k, t):
    rng = np.random.default_rng(7 + E)
    L = rng.standard_normal((6, E))
    G = rng.standard_normal((6, E))
    dL = orc.softtopk_bwd(L, G, k, t)
    h = 1e-6
    num = np.zeros_like(L)
    for j in range(E):
        Lp, Lm = L.copy(), L.copy()
        Lp[:, j] += h; Lm[:, j] -= h
        num[:, j] = ((orc.softtopk_fwd(Lp, k, t) - orc.softtopk_fwd(Lm, k, t)) * G).sum(1) / (2 * h)
    np.testing.assert_allclose(dL, num, rtol=2e-6, atol=2e-8)
    # shift invariance of the forward => gradient sums to zero
    np.testing.assert_allclose(dL.sum(1), 0.0, atol=1e-12)


def test_bwd_k1_is_softmax_jacobian(orc):
    rng = np.random.default_rng(3)
    L = rng.standard_normal((5, 9)); G = rng.standard_normal((5, 9)); t = 2.0
    p = scipy.special.softmax(L / t, axis=1)
    want = p * (G - (G * p).sum(1, keepdims=True)) / t
    np.testing.assert_allclose(orc.softtopk_bwd(L, G, 1, t), want, rtol=1e-12, atol=1e-15)


def test_aux_loss_eq9(orc):
    rng = np.random.default_rng(4)
    T, E, k, lam = 40, 8, 2, 1e-2
    A = rng.random((T, E))
    idx = np.sort(np.argsort(-A, axis=1)[:, :k], axis=1).astype(np.int32)
    P = np.zeros((T, E)); np.put_along_axis(P, idx.astype(np.int64), 1.0, axis=1)
    want = lam / E * (A.mean(0) * P.mean(0)).sum()
    assert abs(orc.aux_loss(A, idx, lam) - want) < 1e-15


def test_aux_loss_grad_matches_finite_differences(orc):
    """Eq. 9 is linear in A, so a central difference of the loss itself is exact up to rounding."""
    rng = np.random.default_rng(5)
    T, E, k, lam = 24, 6, 2, 3e-2
    A = rng.random((T, E))
    idx = np.sort(np.argsort(-A, axis=1)[:, :k], axis=1).astype(np.int32)
    g = orc.aux_loss_grad(idx, T, E, lam)
    assert g.shape == (E,)
    h = 1e-3
    for (i, j) in [(0, 0), (5, 3), (23, 5), (11, 1)]:
        Ap, Am = A.copy(), A.copy()
        Ap[i, j] += h; Am[i, j] -= h
        fd = (orc.aux_loss(Ap, idx, lam) - orc.aux_loss(Am, idx, lam)) / (2 * h)
        assert abs(fd - g[j]) < 1e-12
    # closed form: lambda / (E T^2) * load_j
    load = np.bincount(idx.ravel(), minlength=E)
    np.testing.assert_allclose(g, lam * load / (E * T * T), rtol=1e-14)


# ---- the literal readings of Eq. 6 ("RANKSCALE"); parity unpinned against the paper ---------------------
def test_rankscale_hand_cases(orc):
    """Worked by hand from y_i = p_i * (beta + t * min(rank_i - delta, k)), ranks from 1, ties lowest index first."""
    p = np.array([[0.8, 0.05, 0.1, 0.05]])
    a = np.log(p)
    np.testing.assert_allclose(orc.softtopk_rankscale_fwd(a, 2, 1.0, 0.0, 0), [[0.8, 0.1, 0.2, 0.1]], rtol=1e-14)
    np.testing.assert_allclose(orc.softtopk_rankscale_fwd(a, 2, 1.0, 1.0, 1), [[0.8, 0.15, 0.2, 0.15]], rtol=1e-14)
    np.testing.assert_allclose(orc.softtopk_rankscale_fwd(a, 2, 0.5, 1.0, 1), [[0.8, 0.1, 0.15, 0.1]], rtol=1e-14)
    # the tie rule: equal logits, the lower index ranks first
    q = np.log(np.array([[0.4, 0.4, 0.2]]))
    np.testing.assert_allclose(orc.softtopk_rankscale_fwd(q, 2, 1.0, 0.0, 0), [[0.4, 0.8, 0.4]], rtol=1e-14)


def test_rankscale_special_cases(orc):
    from scipy.special import softmax
    rng = np.random.default_rng(6)
    a = rng.normal(size=(7, 12))
    # t = 0 with base Softmax is the softmax itself (library routine)
    np.testing.assert_allclose(orc.softtopk_rankscale_fwd(a, 3, 0.0, 1.0, 1), softmax(a, axis=1), rtol=1e-13)
    # shift invariance and permutation equivariance
    y = orc.softtopk_rankscale_fwd(a, 3, 0.7, 0.0, 0)
    np.testing.assert_allclose(orc.softtopk_rankscale_fwd(a + 5.0, 3, 0.7, 0.0, 0), y, rtol=1e-12)
    perm = rng.permutation(12)
    np.testing.assert_allclose(orc.softtopk_rankscale_fwd(a[:, perm], 3, 0.7, 0.0, 0), y[:, perm], rtol=1e-12)
    # k = E, (0, 0): every entry is scaled by t * its rank
    ranks = (-a).argsort(1).argsort(1) + 1
    np.testing.assert_allclose(orc.softtopk_rankscale_fwd(a, 12, 2.0, 0.0, 0), softmax(a, axis=1) * 2.0 * ranks, rtol=1e-13)


@pytest.mark.parametrize("beta,delta", [(0.0, 0), (1.0, 1)])
def test_rankscale_bwd_finite_differences(orc, beta, delta):
    rng = np.random.default_rng(8)
    a = rng.normal(size=(3, 9)); g = rng.normal(size=(3, 9))
    k, t, h = 3, 0.8, 1e-6
    got = orc.softtopk_rankscale_bwd(a, g, k, t, beta, delta)
    for (r, l) in [(0, 0), (1, 4), (2, 8), (0, 5)]:
        ap, am = a.copy(), a.copy()
        ap[r, l] += h; am[r, l] -= h
        fd = ((orc.softtopk_rankscale_fwd(ap, k, t, beta, delta) - orc.softtopk_rankscale_fwd(am, k, t, beta, delta)) * g).sum() / (2 * h)
        assert abs(fd - got[r, l]) < 1e-7
    # a softmax Jacobian applied to anything sums to zero over the logits
    np.testing.assert_allclose(got.sum(1), 0.0, atol=1e-14)


# ------------------------------------------------------------------------------------------- IterTopk (Table 2)
def test_itertopk_special_cases_and_invariants(orc):
    rng = np.random.default_rng(21)
    L = rng.normal(size=(40, 12)) * 2.0
    for k in (1, 2, 5, 12):
        Y = orc.itertopk_fwd(L, k)
        np.testing.assert_allclose(Y.sum(axis=1), k, rtol=0, atol=1e-12)          # every level adds a distribution
        np.testing.assert_allclose(orc.itertopk_fwd(L + 3.25, k), Y, rtol=0, atol=1e-11 * np.abs(Y).max() ** 2)   # shift invariance
        perm = rng.permutation(12)
        # (at k = E the recursion overshoots 1 and amplifies rounding: the bar scales with the values)
        np.testing.assert_allclose(orc.itertopk_fwd(L[:, perm], k), Y[:, perm], rtol=0, atol=1e-12 * np.abs(Y).max() ** 2)
    from scipy.special import softmax
    np.testing.assert_allclose(orc.itertopk_fwd(L, 1), softmax(L, axis=1), rtol=0, atol=1e-14)   # k = 1 is Softmax
    # equal logits: every level is uniform over equal weights, so y = k / E
    np.testing.assert_allclose(orc.itertopk_fwd(np.full((1, 8), 0.7), 3), np.full((1, 8), 3 / 8), atol=1e-15)


def test_itertopk_two_experts_closed_form(orc):
    """E = 2, k = 2 by hand: level 1 gives (p, 1-p) with p = softmax; level 2 weights are (1-p, p), and
    (1-p) e^a and p e^b are equal (both are e^a e^b / (e^a + e^b)), so level 2 adds (1/2, 1/2)."""
    for a, b in [(0.3, -1.1), (2.0, 2.0), (-4.0, 1.5)]:
        p = np.exp(a) / (np.exp(a) + np.exp(b))
        Y = orc.itertopk_fwd(np.array([[a, b]]), 2)
        np.testing.assert_allclose(Y, [[p + 0.5, 1.5 - p]], rtol=0, atol=1e-14)
    # E = 3, k = 2, worked with exact fractions for e^x = (4, 2, 2): level 1 = (1/2, 1/4, 1/4); weights (1/2, 3/4, 3/4);
    # w e^x = (2, 3/2, 3/2), sum 5; level 2 = (2/5, 3/10, 3/10); total (9/10, 11/20, 11/20)
    x = np.log(np.array([[4.0, 2.0, 2.0]]))
    np.testing.assert_allclose(orc.itertopk_fwd(x, 2), [[0.9, 0.55, 0.55]], rtol=0, atol=1e-14)


def test_itertopk_backward_against_finite_differences(orc):
    rng = np.random.default_rng(22)
    T, E = 6, 7
    L = rng.normal(size=(T, E)) * 1.5
    G = rng.normal(size=(T, E))
    for k in (1, 2, 4, 7):
        dL = orc.itertopk_bwd(L, G, k)
        h = 1e-6
        num = np.zeros_like(L)
        for j in range(E):
            Lp, Lm = L.copy(), L.copy()
            Lp[:, j] += h; Lm[:, j] -= h
            num[:, j] = ((orc.itertopk_fwd(Lp, k) - orc.itertopk_fwd(Lm, k)) * G).sum(axis=1) / (2 * h)
        np.testing.assert_allclose(dL, num, rtol=1e-7, atol=2e-8)
        np.testing.assert_allclose(dL.sum(axis=1), 0, atol=1e-10 * max(1.0, np.abs(dL).max()))   # shift invariance of the forward
