"""Pins for the oracle's assignment solvers (Eq. 7-8, Table 1) and index/dispatch/combine."""
import itertools

import numpy as np
import pytest
import scipy.optimize


def _rand_keys(rng, T, E, lo=-50, hi=50):
    return rng.integers(lo, hi, size=(T, E)).astype(np.int64)


def _check_invariants(idx, load, T, E, k, C):
    assert idx.shape == (T, k)
    assert (idx >= 0).all() and (idx < E).all()
    assert (np.diff(idx, axis=1) > 0).all()                 # k distinct experts, ascending
    cnt = np.bincount(idx.ravel(), minlength=E)
    np.testing.assert_array_equal(cnt, load)                # flow conservation at the experts
    assert (load <= C).all()
    assert load.sum() == T * k                              # maximum flow: every token fully served


# ---------------------------------------------------------------- brute force
@pytest.mark.parametrize("T,E,k,C", [(6, 3, 2, 4), (8, 4, 2, 4), (7, 4, 2, 4), (5, 4, 3, 4),
                                      (8, 4, 1, 2), (6, 4, 2, 5), (8, 3, 1, 3), (4, 4, 4, 4)])
def test_solvers_reach_bruteforce_optimum(orc, T, E, k, C):
    rng = np.random.default_rng(T * 1000 + E * 100 + k * 10 + C)
    for trial in range(6):
        # narrow key ranges on odd trials force many ties
        w = _rand_keys(rng, T, E, -3, 3) if trial % 2 else _rand_keys(rng, T, E, -1000, 1000)
        best, n_opt, bidx = orc.flow_bruteforce(w, k, C)
        assert best == orc.primal_value(w, bidx)
        for solver in (orc.flow_ssp, orc.flow_condensed):
            idx, load, _ = solver(w, k, C)
            _check_invariants(idx, load, T, E, k, C)
            assert orc.primal_value(w, idx) == best, solver.__name__
            res, prices = orc.flow_certificate(w, idx, C)
            assert res == (2 if n_opt == 1 else 1)
            # strong duality, exact in integers
            assert (prices >= 0).all()
            assert orc.dual_value(w, prices, k, C) == best
            if n_opt == 1:
                np.testing.assert_array_equal(idx, bidx)


def test_bruteforce_against_python_enumeration(orc):
    # the enumerator itself, restated with itertools on a 4-token case
    rng = np.random.default_rng(5)
    T, E, k, C = 4, 4, 2, 2
    w = _rand_keys(rng, T, E)
    subsets = list(itertools.combinations(range(E), k))
    best, count = None, 0
    for choice in itertools.product(subsets, repeat=T):
        load = np.zeros(E, int)
        for s in choice:
            load[list(s)] += 1
        if (load > C).any():
            continue
        tot = sum(int(w[i, list(s)].sum()) for i, s in enumerate(choice))
        if best is None or tot > best:
            best, count = tot, 1
        elif tot == best:
            count += 1
    b, n, _ = orc.flow_bruteforce(w, k, C)
    assert (b, n) == (best, count)


def test_certificate_rejects_suboptimal_and_infeasible(orc):
    rng = np.random.default_rng(11)
    T, E, k, C = 8, 4, 2, 4
    w = _rand_keys(rng, T, E, -1000, 1000)
    idx, load, _ = orc.flow_ssp(w, k, C)
    assert orc.flow_certificate(w, idx, C)[0] >= 1
    # swap the experts of two tokens in a way that keeps loads but lowers the score
    worse = None
    for i, j in itertools.combinations(range(T), 2):
        for a in range(k):
            for b in range(k):
                ea, eb = idx[i, a], idx[j, b]
                if ea == eb or eb in idx[i] or ea in idx[j]:
                    continue
                cand = idx.copy(); cand[i, a] = eb; cand[j, b] = ea
                cand.sort(axis=1)
                if orc.primal_value(w, cand) < orc.primal_value(w, idx):
                    worse = cand
    assert worse is not None
    assert orc.flow_certificate(w, worse, C)[0] == 0
    # over capacity / duplicate expert -> invariant failure
    bad = idx.copy(); bad[:, 0] = 0; bad[:, 1] = 1
    assert orc.flow_certificate(w, bad, C)[0] == -1
    dup = idx.copy(); dup[0, 1] = dup[0, 0]
    assert orc.flow_certificate(w, dup, C)[0] == -1


# ---------------------------------------------------------------- reductions to textbook routines
def test_loose_capacity_is_per_token_topk(orc):
    rng = np.random.default_rng(12)
    T, E, k = 60, 8, 3
    w = rng.permutation(T * E).reshape(T, E).astype(np.int64)   # all keys distinct
    want = np.sort(np.argsort(-w, axis=1)[:, :k], axis=1)
    for solver in (orc.flow_ssp, orc.flow_condensed):
        idx, load, _ = solver(w, k, T)
        np.testing.assert_array_equal(idx, want)


@pytest.mark.parametrize("T,E,C", [(12, 3, 4), (20, 4, 5), (15, 4, 5)])
def test_k1_is_linear_assignment(orc, T, E, C):
    # k = 1: a T x (E*C) assignment problem with each expert's column repeated C times
    rng = np.random.default_rng(T + E)
    w = _rand_keys(rng, T, E, -500, 500)
    cost = -np.repeat(w, C, axis=1)
    r, c = scipy.optimize.linear_sum_assignment(cost)
    want = -cost[r, c].sum()
    for solver in (orc.flow_ssp, orc.flow_condensed):
        idx, load, _ = solver(w, 1, C)
        _check_invariants(idx, load, T, E, 1, C)
        assert orc.primal_value(w, idx) == want


def test_k2_equals_min_cost_flow_via_lp(orc):
    # the flow LP is totally unimodular: its LP optimum (scipy linprog) equals the integer optimum
    rng = np.random.default_rng(13)
    T, E, k, C = 16, 4, 2, 8
    w = _rand_keys(rng, T, E, -100, 100)
    A_eq = np.zeros((T, T * E)); A_ub = np.zeros((E, T * E))
    for i in range(T):
        A_eq[i, i * E:(i + 1) * E] = 1
    for e in range(E):
        A_ub[e, e::E] = 1
    res = scipy.optimize.linprog(-w.ravel().astype(float), A_ub=A_ub, b_ub=np.full(E, C), A_eq=A_eq,
                                 b_eq=np.full(T, k), bounds=(0, 1), method="highs")
    assert res.status == 0
    idx, load, _ = orc.flow_ssp(w, k, C)
    assert orc.primal_value(w, idx) == round(-res.fun)


# ---------------------------------------------------------------- medium sizes: solver agreement + certificate
@pytest.mark.parametrize("T,E,k,cf", [(512, 8, 2, 1.0), (256, 16, 4, 1.0), (300, 8, 2, 1.25), (384, 12, 3, 1.5)])
def test_textbook_and_condensed_agree(orc, T, E, k, cf):
    rng = np.random.default_rng(T + E + k)
    A = orc.softtopk_fwd(rng.standard_normal((T, E)), k, 1.0)
    w = orc.keys_from_scores(A)
    C = orc.capacity(T, k, E, cf)
    i1, l1, fv = orc.flow_ssp(w, k, C)
    i2, l2, _ = orc.flow_condensed(w, k, C)
    assert fv == T * k
    _check_invariants(i1, l1, T, E, k, C)
    _check_invariants(i2, l2, T, E, k, C)
    assert orc.primal_value(w, i1) == orc.primal_value(w, i2)
    r1, p1 = orc.flow_certificate(w, i1, C)
    r2, p2 = orc.flow_certificate(w, i2, C)
    assert r1 >= 1 and r2 >= 1
    assert orc.dual_value(w, p1, k, C) == orc.primal_value(w, i1)
    if r1 == 2:
        np.testing.assert_array_equal(i1, i2)
    if cf == 1.0 and (T * k) % E == 0:
        assert (l1 == C).all()                       # exact flow fills every expert (Sec. 4.5 load ratio 1)


def test_integer_keys_and_unique_optimum(orc):
    rng = np.random.default_rng(21)
    T, E, k = 256, 8, 2
    L = rng.standard_normal((T, E)).astype(np.float32)
    w, q = orc.keys_from_logits(L, k, 11, seed=0)
    S = orc.tiebreak_shift(T, k)
    assert S == 20 + 9
    # q is round-to-nearest-even of L*2^11, clamped to int16
    want_q = np.clip(np.rint(L.astype(np.float64) * 2048), -32768, 32767).astype(np.int16)
    np.testing.assert_array_equal(q, want_q)
    r = w - (q.astype(np.int64) << S)
    assert (r >= 0).all() and (r < (1 << 20)).all()
    assert len(np.unique(r)) > 0.99 * r.size * (1 - r.size / 2 ** 21)   # hash spreads
    # a different seed gives a different perturbation, the same q
    w2, q2 = orc.keys_from_logits(L, k, 11, seed=1)
    np.testing.assert_array_equal(q, q2)
    assert (w2 != w).mean() > 0.99
    C = orc.capacity(T, k, E, 1.0)
    idx, load, _ = orc.flow_ssp(w, k, C)
    res, _ = orc.flow_certificate(w, idx, C)
    assert res == 2
    # the perturbation never outweighs one step of q: the q-only score is optimal too
    wq = q.astype(np.int64)
    iq, _, _ = orc.flow_ssp(wq, k, C)
    assert orc.primal_value(wq, idx) == orc.primal_value(wq, iq)


def test_murmur_finaliser_known_values(orc):
    # fmix32 is a bijection with fmix32(0) = 0; check the key of entry (0,0) with seed 0 and
    # two values computed by hand from the published finaliser
    def fmix32(h):
        h ^= h >> 16; h = (h * 0x85EBCA6B) & 0xFFFFFFFF
        h ^= h >> 13; h = (h * 0xC2B2AE35) & 0xFFFFFFFF
        h ^= h >> 16
        return h
    L = np.zeros((2, 4), np.float32)
    w, _ = orc.keys_from_logits(L, 1, 11, seed=3)
    for i in range(2):
        for j in range(4):
            want = fmix32((i * 4 + j + 3 * 0x9E3779B9) & 0xFFFFFFFF) >> 12
            assert w[i, j] == want
    w0, _ = orc.keys_from_logits(L, 1, 11, seed=0)
    assert w0[0, 0] == 0


def test_infeasible_is_reported(orc):
    w = np.zeros((8, 4), np.int64)
    with pytest.raises(ValueError):
        orc.flow_ssp(w, 2, 3)       # 4*3 < 16
    with pytest.raises(ValueError):
        orc.flow_condensed(w, 2, 3)


def test_negative_scores_still_fill_k(orc):
    # maximum flow comes first: tokens take k experts even when every key is negative
    rng = np.random.default_rng(30)
    w = -np.abs(_rand_keys(rng, 12, 4, 1, 100))
    idx, load, fv = orc.flow_ssp(w, 2, 6)
    assert fv == 24
    _check_invariants(idx, load, 12, 4, 2, 6)


# ---------------------------------------------------------------- index build / dispatch / combine
def test_index_dispatch_combine(orc):
    rng = np.random.default_rng(40)
    T, E, k, d = 96, 8, 2, 24
    C = orc.capacity(T, k, E, 1.25)
    A = orc.softtopk_fwd(rng.standard_normal((T, E)), k, 1.0)
    idx, load, _ = orc.flow_condensed(orc.keys_from_scores(A), k, C)
    slot_idx, slot_token, load2 = orc.index_build(idx, E, C)
    np.testing.assert_array_equal(load, load2)
    # mutual inverses, ascending token order inside each expert, -1 padding behind the load
    for e in range(E):
        row = slot_token[e]
        assert (row[:load[e]] >= 0).all() and (row[load[e]:] == -1).all()
        assert (np.diff(row[:load[e]]) > 0).all()
    for i in range(T):
        for c in range(k):
            assert slot_token[idx[i, c], slot_idx[i, c]] == i
    H = rng.standard_normal((T, d)).astype(np.float32)
    xd = orc.dispatch(H, slot_token)
    assert xd.dtype == np.float32 and xd.shape == (E, C, d)
    for e in range(E):
        np.testing.assert_array_equal(xd[e, :load[e]], H[slot_token[e, :load[e]]])
        assert (xd[e, load[e]:] == 0).all()
    # 2-byte rows move bit-exactly too
    H16 = rng.integers(0, 65536, size=(T, d)).astype(np.uint16)
    xd16 = orc.dispatch(H16, slot_token)
    np.testing.assert_array_equal(xd16[idx[5, 1], slot_idx[5, 1]], H16[5])
    # identity experts: Y_i = (sum of the token's gate weights) * H_i
    gw = orc.gate_weights(A, idx)
    Y = orc.combine(xd, idx, slot_idx, gw)
    np.testing.assert_allclose(Y, gw.sum(1, keepdims=True) * H.astype(np.float64), rtol=1e-13)
    # unit weights = adjoint of dispatch: <dispatch(x), y> = <x, combine_unit(y)>
    Yb = rng.standard_normal((E, C, d))
    lhs = (xd.astype(np.float64) * Yb).sum()
    rhs = (H.astype(np.float64) * orc.combine(Yb, idx, slot_idx, None)).sum()
    assert abs(lhs - rhs) < 1e-9 * max(1.0, abs(lhs))
    with pytest.raises(ValueError):
        orc.index_build(idx, E, int(load.max()) - 1)


def test_backward_chain_finite_differences(orc):
    rng = np.random.default_rng(41)
    T, E, k, d, t = 24, 6, 2, 10, 1.5
    C = orc.capacity(T, k, E, 1.0)
    H = rng.standard_normal((T, d)); W = rng.standard_normal((d, E)) / np.sqrt(d)
    yexp = rng.standard_normal((E, C, d)); dY = rng.standard_normal((T, d))
    L = orc.gate(H, W)
    A = orc.softtopk_fwd(L, k, t)
    idx, _, _ = orc.flow_ssp(orc.keys_from_scores(A), k, C)
    slot_idx, slot_token, _ = orc.index_build(idx, E, C)

    def loss(Hx, Wx, yx):
        Ax = orc.softtopk_fwd(orc.gate(Hx, Wx), k, t)
        return (orc.combine(yx, idx, slot_idx, orc.gate_weights(Ax, idx)) * dY).sum()   # P held fixed

    gw = orc.gate_weights(A, idx)
    dyexp, dgw = orc.combine_bwd(dY, yexp, idx, slot_idx, gw)
    G = np.zeros((T, E)); np.put_along_axis(G, idx.astype(np.int64), dgw, axis=1)
    dL = orc.softtopk_bwd(L, G, k, t)
    dW, dH = orc.gate_bwd(H, W, dL)
    h = 1e-6
    for (arr, grad, name) in ((W, dW, "W"), (H, dH, "H"), (yexp, dyexp, "yexp")):
        flat = arr.reshape(-1)
        for pos in rng.choice(flat.size, 12, replace=False):
            old = flat[pos]
            flat[pos] = old + h; fp = loss(H, W, yexp)
            flat[pos] = old - h; fm = loss(H, W, yexp)
            flat[pos] = old
            num = (fp - fm) / (2 * h)
            assert abs(num - grad.reshape(-1)[pos]) < 1e-6 * max(1.0, abs(num)), name
    # padding rows of dyexp carry no gradient; gate_bwd against library matmuls
    assert (dyexp[slot_token < 0] == 0).all()
    np.testing.assert_allclose(dW, H.T @ dL, atol=1e-12)
    np.testing.assert_allclose(dH, dL @ W.T, atol=1e-12)


def test_float_keys_round_to_nearest_even_on_the_2_pow_minus_40_grid(orc):
    """mso_keys_from_scores against numpy's rint (an independent library routine), half-way cases included:
    a plausible mistake (truncation, round-half-up, another scale) fails one of them."""
    rng = np.random.default_rng(3)
    A = rng.random((37, 11)) * 3.0
    np.testing.assert_array_equal(orc.keys_from_scores(A), np.rint(A * 2.0 ** 40).astype(np.int64))
    # exact half-way points (odd multiples of 2^-41) must go to the even neighbour, both signs
    m = np.array([1, 3, 5, 7, 2 ** 20 + 1, 2 ** 30 + 3, -1, -3, -5], dtype=np.float64)
    half = m * 2.0 ** -41
    want = np.array([0, 2, 2, 4, 2 ** 19, 2 ** 29 + 2, 0, -2, -2], dtype=np.int64)
    np.testing.assert_array_equal(orc.keys_from_scores(half.reshape(1, -1))[0], want)
    # scale: one unit of the key is 2^-40 of score, so 1.0 -> 2^40 and 2^-40 -> 1
    np.testing.assert_array_equal(orc.keys_from_scores(np.array([[1.0, 2.0 ** -40, 0.75]])),
                                  np.array([[2 ** 40, 1, 3 * 2 ** 38]], dtype=np.int64))


def test_hashed_float_keys_hand_values_and_bounds(orc):
    """The position hash of the documented float-mode keys: hand-computed values of
    ((i*E + j) * 2654435761 mod 2^32) >> 20 at a few positions, its range, that it depends on the position
    only, and that it never changes which of two different float scores is larger."""
    Z = np.zeros((3, 4))
    h = orc.keys_from_scores_hashed(Z)
    # position 0: 0; 1: 2654435761 >> 20 = 2531; 2: (5308871522 - 2^32 = 1013904226) >> 20 = 966;
    # 3: (7963307283 - 2^32 = 3668339987) >> 20 = 3498; 5: (13272178805 - 3*2^32 = 387276917) >> 20 = 369
    assert h[0, 0] == 0 and h[0, 1] == 2531 and h[0, 2] == 966 and h[0, 3] == 3498 and h[1, 1] == 369
    rng = np.random.default_rng(5)
    A = rng.random((64, 16)).astype(np.float32).astype(np.float64)
    w0, w1 = orc.keys_from_scores(A), orc.keys_from_scores_hashed(A)
    d = w1 - w0
    assert d.min() >= 0 and d.max() < 4096
    np.testing.assert_array_equal(d, orc.keys_from_scores_hashed(np.zeros_like(A)))      # position only
    # the position is the row-major flat index i*E + j (a transposed index would give other values)
    np.testing.assert_array_equal(d.reshape(-1), orc.keys_from_scores_hashed(np.zeros((1, 64 * 16)))[0])
    assert not np.array_equal(d.T.reshape(-1), d.reshape(-1))
    # two different fp32 scores differ by at least one ulp, which is >= 2^-24 relative, i.e. >= 2^16 key units
    # for scores >= 2^-0: the 12-bit hash cannot reorder them
    order0 = np.argsort(-w0, axis=1, kind="stable")
    order1 = np.argsort(-w1, axis=1, kind="stable")
    distinct = np.diff(np.sort(A, axis=1), axis=1).min() > 0
    assert distinct and np.array_equal(order0, order1)
    # and the optimum of a small problem moves by less than 4e-9 per chosen pair
    T, E, k, C = 6, 4, 2, 3
    S = rng.random((T, E)).astype(np.float32).astype(np.float64)
    i0, _, _ = orc.flow_ssp(orc.keys_from_scores(S), k, C)
    i1, _, _ = orc.flow_ssp(orc.keys_from_scores_hashed(S), k, C)
    assert abs(orc.total_score(S, i0) - orc.total_score(S, i1)) < 4e-9 * T * k


# ------------------------------------------------------------------------------------------- iterative rerouting
def _reroute_by_hand(A, k, C):
    """Independent restatement with Python lists and sorting (no shared code with the C routine)."""
    T, E = A.shape
    order = [sorted(range(E), key=lambda j: (-A[i, j], j))[:k] for i in range(T)]
    load = [0] * E
    held = [set() for _ in range(T)]
    dropped = []
    for r in range(k):
        for i in range(T):
            e = order[i][r]
            if load[e] < C:
                load[e] += 1; held[i].add(e)
            else:
                dropped.append((i, r))
    empty = 0
    for i, r in sorted(dropped):
        free = [j for j in range(E) if load[j] < C and j not in held[i]]
        if not free:
            empty += 1
            continue
        e = min(free, key=lambda j: (-A[i, j], j))
        load[e] += 1; held[i].add(e)
    idx = np.full((T, k), -1, np.int32)
    for i in range(T):
        s = sorted(held[i])
        idx[i, :len(s)] = s
    return idx, np.array(load, np.int32), len(dropped), empty


def test_iterative_reroute_small_cases_and_invariants(orc):
    rng = np.random.default_rng(31)
    for (T, E, k, C) in [(12, 4, 2, 6), (40, 8, 2, 10), (33, 5, 3, 20), (64, 16, 4, 16), (9, 3, 3, 9), (20, 4, 2, 7)]:
        A = rng.random((T, E)).astype(np.float32).astype(np.float64)
        idx, load, nd, ne = orc.iterative_reroute(A, k, C)
        widx, wload, wnd, wne = _reroute_by_hand(A, k, C)
        np.testing.assert_array_equal(idx, widx); np.testing.assert_array_equal(load, wload)
        assert (nd, ne) == (wnd, wne)
        assert (load <= C).all() and load.sum() == T * k - ne
        filled = idx >= 0
        assert np.array_equal(np.bincount(idx[filled], minlength=E), load)
        for i in range(T):                                   # distinct experts, ascending, empty slots last
            row = idx[i][idx[i] >= 0]
            assert (np.diff(row) > 0).all() and (idx[i][len(row):] == -1).all()
    # loose capacity: nothing is dropped and the result is plain top-k
    A = rng.random((50, 8))
    idx, load, nd, ne = orc.iterative_reroute(A, 3, 50)
    assert nd == 0 and ne == 0
    np.testing.assert_array_equal(idx, np.sort(np.argsort(-A, axis=1, kind="stable")[:, :3], axis=1))


def test_iterative_reroute_hand_case_and_suboptimality(orc):
    """Three tokens, two experts, k = 1, C = 2, affinities chosen so that level 1 overloads expert 0:
    tokens 0 and 1 take it, token 2 is dropped and rerouted to expert 1.  The exact flow would instead move
    the token that loses least (token 1): greedy rerouting is feasible but not optimal (Sec. 3.2's trade-off)."""
    A = np.array([[0.9, 0.1], [0.6, 0.5], [0.8, 0.0]])
    idx, load, nd, ne = orc.iterative_reroute(A, 1, 2)
    np.testing.assert_array_equal(idx, [[0], [0], [1]])
    np.testing.assert_array_equal(load, [2, 1])
    assert (nd, ne) == (1, 0)
    oidx, _, _ = orc.flow_ssp(orc.keys_from_scores(A), 1, 2)
    np.testing.assert_array_equal(oidx, [[0], [1], [0]])
    assert orc.total_score(A, oidx) > orc.total_score(A, idx)
    # tied affinities go to the lowest expert index at both stages
    A = np.array([[0.5, 0.5, 0.5], [0.5, 0.5, 0.5], [0.5, 0.5, 0.5]])
    idx, load, nd, ne = orc.iterative_reroute(A, 1, 1)
    np.testing.assert_array_equal(idx, [[0], [1], [2]])


# ------------------------------------------------------------------------------------------- Algorithm 1
def test_alg1_first_stage_is_plain_top1_and_residuals(orc):
    rng = np.random.default_rng(41)
    T, E, C = 60, 6, 20
    A = rng.random((T, E))
    first, second, resid, over, dropped, plan = orc.alg1_top1_sinkhorn(A, C, 0.05, 2000, want_plan=True)
    np.testing.assert_array_equal(first, A.argmax(axis=1))                       # step 4: one-hot of the arg-max
    cnt = np.bincount(first, minlength=E)
    np.testing.assert_array_equal(resid, np.maximum(0, C - cnt))                 # step 6
    assert over == np.maximum(0, cnt - C).sum()
    # the plan: masked pairs carry nothing, rows sum to one, capped columns stay within the residual capacity
    assert (plan[np.arange(T), first] == 0).all()
    np.testing.assert_allclose(plan.sum(axis=1), 1.0, atol=1e-12)
    assert (plan.sum(axis=0) <= resid * (1 + 1e-3) + 1e-9).all()
    # rounding: the second expert differs from the first, is the plan's arg-max unless dropped, and no expert
    # gets more seconds than it has room for
    keep = second >= 0
    assert (second[keep] != first[keep]).all()
    np.testing.assert_array_equal(second[keep], plan.argmax(axis=1)[keep])
    assert (np.bincount(second[keep], minlength=E) <= resid).all()
    assert dropped == (~keep).sum()
    # ties in the first stage go to the lowest index
    f2, *_ = orc.alg1_top1_sinkhorn(np.full((4, 3), 0.5), 4, 0.1, 3)
    np.testing.assert_array_equal(f2, 0)


def test_alg1_with_loose_capacity_is_plain_top2(orc):
    rng = np.random.default_rng(42)
    A = rng.random((80, 8))
    first, second, resid, over, dropped = orc.alg1_top1_sinkhorn(A, 80, 0.07, 10)   # nobody is ever capped
    order = np.argsort(-A, axis=1, kind="stable")
    np.testing.assert_array_equal(first, order[:, 0])
    np.testing.assert_array_equal(second, order[:, 1])
    assert over == 0 and dropped == 0


def test_alg1_second_stage_tends_to_the_lp_optimum(orc):
    """Small regulariser, many iterations: the plan's value approaches the optimum of the residual transport
    problem (rows = 1, columns <= residual capacity, masked pairs excluded), computed by scipy's LP solver."""
    from scipy.optimize import linprog
    rng = np.random.default_rng(43)
    T, E, C = 10, 4, 5
    A = rng.random((T, E))
    first, second, resid, over, dropped, plan = orc.alg1_top1_sinkhorn(A, C, 0.01, 4000, want_plan=True)
    cost = -A.copy(); cost[np.arange(T), first] = 0.0
    bounds = [(0, 0) if j == first[i] else (0, None) for i in range(T) for j in range(E)]
    A_eq = np.zeros((T, T * E)); A_ub = np.zeros((E, T * E))
    for i in range(T):
        A_eq[i, i * E:(i + 1) * E] = 1
    for j in range(E):
        A_ub[j, j::E] = 1
    res = linprog(cost.reshape(-1), A_ub=A_ub, b_ub=resid.astype(float), A_eq=A_eq, b_eq=np.ones(T), bounds=bounds)
    assert res.status == 0
    got = (plan * A).sum()
    # from above only by what the not yet fully converged column caps allow; from below by the entropic gap
    # (at most eps * log E per token)
    assert got <= -res.fun + 1e-3 and got >= -res.fun - 0.02 * T
    np.testing.assert_allclose(plan.sum(axis=0), np.minimum(plan.sum(axis=0), resid), atol=1e-3)
