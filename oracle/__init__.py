"""ctypes front end of the CPU oracle (oracle/maxscore_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
CPU-baseline leg of bench.py.  The CUDA package never imports this module and
this module never imports the CUDA package.

Every function takes and returns numpy arrays; floating-point inputs are
converted to float64 here (exactly, from fp32 or bf16 values the caller has
already widened), integers to the widths the C side declares.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from fractions import Fraction

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "maxscore_oracle.c")
_LIB = os.path.join(_HERE, "libmaxscore_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP on the per-token loops)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=gnu11", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.mso_capacity.restype = C.c_int64
        _lib.mso_capacity.argtypes = [C.c_int64] * 5
        _lib.mso_feasible.restype = C.c_int
        _lib.mso_feasible.argtypes = [C.c_int64] * 4
        _lib.mso_aux_loss.restype = C.c_double
    return _lib


def threads() -> int:
    """Number of OpenMP threads the per-token loops use."""
    n = os.environ.get("OMP_NUM_THREADS")
    return int(n) if n else (os.cpu_count() or 1)


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _i64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int64))


I64 = C.c_int64


def capacity(T: int, k: int, E: int, capacity_factor) -> int:
    """C = ceil(cf*T*k/E), exact: cf is turned into a fraction first (Sec. 2.3)."""
    cf = Fraction(capacity_factor).limit_denominator(1 << 20)
    return int(lib().mso_capacity(T, k, E, cf.numerator, cf.denominator))


def feasible(T: int, k: int, E: int, Cap: int) -> bool:
    return bool(lib().mso_feasible(T, k, E, Cap))


def gate(H, W, bias=None) -> np.ndarray:
    """Eq. 2: L = H @ W (+ bias), W given as [d, E]; float64 result."""
    H, W = _f64(H), _f64(W)
    T, d = H.shape
    E = W.shape[1]
    assert W.shape[0] == d
    L = np.empty((T, E), np.float64)
    b = _f64(bias) if bias is not None else None
    lib().mso_gate(I64(T), I64(d), I64(E), _p(H), _p(W), _p(b) if b is not None else None, _p(L))
    return L


def softtopk_fwd(L, k: int, t: float) -> np.ndarray:
    """Eq. 6 (ITERMASK reading); float64 affinities A[T, E]."""
    L = _f64(L)
    T, E = L.shape
    A = np.empty_like(L)
    rc = lib().mso_softtopk_fwd(I64(T), I64(E), I64(k), C.c_double(t), _p(L), _p(A))
    if rc:
        raise ValueError("softtopk_fwd: bad arguments")
    return A


def softtopk_bwd(L, G, k: int, t: float) -> np.ndarray:
    """dL = J^T G for Eq. 6 with the masks held constant."""
    L, G = _f64(L), _f64(G)
    T, E = L.shape
    dL = np.empty_like(L)
    rc = lib().mso_softtopk_bwd(I64(T), I64(E), I64(k), C.c_double(t), _p(L), _p(G), _p(dL))
    if rc:
        raise ValueError("softtopk_bwd: bad arguments")
    return dL


def softtopk_rankscale_fwd(L, k: int, t: float, beta: float, delta: int) -> np.ndarray:
    """The literal readings of Eq. 6: y = softmax(a) * (beta + t * min(rank - delta, k)).  Parity unpinned
    against the paper (it prints no value that separates the readings)."""
    L = _f64(L)
    T, E = L.shape
    A = np.empty_like(L)
    rc = lib().mso_softtopk_rankscale_fwd(I64(T), I64(E), I64(k), C.c_double(t), C.c_double(beta), I64(delta),
                                          _p(L), _p(A))
    if rc:
        raise ValueError("softtopk_rankscale_fwd: bad arguments")
    return A


def softtopk_rankscale_bwd(L, G, k: int, t: float, beta: float, delta: int) -> np.ndarray:
    L, G = _f64(L), _f64(G)
    T, E = L.shape
    dL = np.empty_like(L)
    rc = lib().mso_softtopk_rankscale_bwd(I64(T), I64(E), I64(k), C.c_double(t), C.c_double(beta), I64(delta),
                                          _p(L), _p(G), _p(dL))
    if rc:
        raise ValueError("softtopk_rankscale_bwd: bad arguments")
    return dL


def itertopk_fwd(L, k: int) -> np.ndarray:
    """IterTopk of Table 2: y^(l) = y^(l-1) + g(x; 1 - y^(l-1)), g(x; w) = w e^x / sum(w e^x), y^(0) = 0."""
    L = _f64(L)
    T, E = L.shape
    A = np.empty_like(L)
    if lib().mso_itertopk_fwd(I64(T), I64(E), I64(k), _p(L), _p(A)):
        raise ValueError("itertopk_fwd: bad arguments")
    return A


def itertopk_bwd(L, G, k: int) -> np.ndarray:
    """dL = J^T G for IterTopk."""
    L, G = _f64(L), _f64(G)
    T, E = L.shape
    dL = np.empty_like(L)
    if lib().mso_itertopk_bwd(I64(T), I64(E), I64(k), _p(L), _p(G), _p(dL)):
        raise ValueError("itertopk_bwd: bad arguments")
    return dL


def alg1_top1_sinkhorn(A, Cap: int, eps: float, iters: int, want_plan: bool = False):
    """Algorithm 1 (top-2): top-1, then capped Sinkhorn on the residual problem and argmax rounding.
    Returns (first [T], second [T] with -1 = dropped, resid [E], top-1 pairs beyond Cap, seconds dropped[, plan])."""
    A = _f64(A)
    T, E = A.shape
    first = np.empty(T, np.int32); second = np.empty(T, np.int32)
    resid = np.empty(E, np.int64); counts = np.zeros(2, np.int64)
    plan = np.empty((T, E), np.float64) if want_plan else None
    rc = lib().mso_alg1_top1_sinkhorn(I64(T), I64(E), I64(Cap), _p(A), C.c_double(eps), I64(iters), _p(first), _p(second),
                                      _p(plan) if want_plan else None, _p(resid), _p(counts))
    if rc:
        raise ValueError("alg1_top1_sinkhorn: bad arguments")
    out = (first, second, resid, int(counts[0]), int(counts[1]))
    return out + (plan,) if want_plan else out


def iterative_reroute(A, k: int, Cap: int):
    """Top-k with capacity, then greedy rerouting of the dropped pairs (Sec. 2.3).  Returns
    (expert_idx [T,k] ascending with -1 last, load [E], pairs dropped in stage 1, slots left empty)."""
    A = _f64(A)
    T, E = A.shape
    idx = np.empty((T, k), np.int32)
    load = np.empty(E, np.int32)
    counts = np.zeros(2, np.int64)
    if lib().mso_iterative_reroute(I64(T), I64(E), I64(k), I64(Cap), _p(A), _p(idx), _p(load), _p(counts)):
        raise ValueError("iterative_reroute: bad arguments")
    return idx, load, int(counts[0]), int(counts[1])


def keys_from_scores(A) -> np.ndarray:
    """Fixed-point keys rne(A * 2^40) as int64."""
    A = _f64(A)
    w = np.empty(A.shape, np.int64)
    lib().mso_keys_from_scores(I64(A.size), _p(A), _p(w))
    return w


def keys_from_scores_hashed(A) -> np.ndarray:
    """Float-mode keys as the library documents them: rne(A * 2^40) plus the 12-bit position hash
    ((i*E + j) * 2654435761 mod 2^32) >> 20."""
    A = _f64(A)
    T, E = A.shape
    w = np.empty(A.shape, np.int64)
    lib().mso_keys_from_scores_hashed(I64(T), I64(E), _p(A), _p(w))
    return w


def tiebreak_shift(T: int, k: int) -> int:
    return int(lib().mso_tiebreak_shift(I64(T), I64(k)))


def keys_from_logits(L32, k: int, quant_shift: int, seed: int):
    """Integer mode keys w = q*2^S + r; returns (w int64 [T,E], q int16 [T,E])."""
    L32 = np.ascontiguousarray(np.asarray(L32, dtype=np.float32))
    T, E = L32.shape
    w = np.empty((T, E), np.int64)
    q = np.empty((T, E), np.int16)
    lib().mso_keys_from_logits(I64(T), I64(E), I64(k), _p(L32), C.c_int(quant_shift),
                               C.c_uint32(seed & 0xFFFFFFFF), _p(w), _p(q))
    return w, q


def flow_ssp(w, k: int, Cap: int):
    """Eq. 7-8 on Table 1's network by textbook successive shortest paths (SPFA).

    Returns (expert_idx int32 [T,k] ascending, load int32 [E], flow_value)."""
    w = _i64(w)
    T, E = w.shape
    idx = np.empty((T, k), np.int32)
    load = np.empty(E, np.int32)
    fv = I64(0)
    rc = lib().mso_flow_ssp(I64(T), I64(E), I64(k), I64(Cap), _p(w), _p(idx), _p(load), C.byref(fv))
    if rc:
        raise ValueError(f"flow_ssp: status {rc}")
    return idx, load, int(fv.value)


def flow_condensed(w, k: int, Cap: int):
    """Same optimum as flow_ssp, path search on the expert-level residual graph."""
    w = _i64(w)
    T, E = w.shape
    idx = np.empty((T, k), np.int32)
    load = np.empty(E, np.int32)
    na = I64(0)
    rc = lib().mso_flow_condensed(I64(T), I64(E), I64(k), I64(Cap), _p(w), _p(idx), _p(load), C.byref(na))
    if rc:
        raise ValueError(f"flow_condensed: status {rc}")
    return idx, load, int(na.value)


def flow_bruteforce(w, k: int, Cap: int):
    """Enumerate all assignments (T<=8, E<=4). Returns (best_total, n_optimal, expert_idx)."""
    w = _i64(w)
    T, E = w.shape
    idx = np.empty((T, k), np.int32)
    best, cnt = I64(0), I64(0)
    rc = lib().mso_flow_bruteforce(I64(T), I64(E), I64(k), I64(Cap), _p(w), C.byref(best),
                                   C.byref(cnt), _p(idx))
    if rc:
        raise ValueError(f"flow_bruteforce: status {rc}")
    return int(best.value), int(cnt.value), idx


def flow_certificate(w, expert_idx, Cap: int):
    """Check an assignment: returns (result, prices).

    result: -1 invariants broken, 0 not optimal, 1 optimal (not unique), 2 uniquely optimal."""
    w = _i64(w)
    T, E = w.shape
    idx = _i32(expert_idx)
    k = idx.shape[1]
    prices = np.zeros(E, np.int64)
    r = lib().mso_flow_certificate(I64(T), I64(E), I64(k), I64(Cap), _p(w), _p(idx), _p(prices))
    return int(r), prices


def _i128(hi, lo) -> int:
    return (int(hi.value) << 64) + int(lo.value)


def dual_value(w, prices, k: int, Cap: int) -> int:
    w, p = _i64(w), _i64(prices)
    T, E = w.shape
    hi, lo = I64(0), C.c_uint64(0)
    lib().mso_dual_value(I64(T), I64(E), I64(k), I64(Cap), _p(w), _p(p), C.byref(hi), C.byref(lo))
    return _i128(hi, lo)


def primal_value(w, expert_idx) -> int:
    w, idx = _i64(w), _i32(expert_idx)
    T, E = w.shape
    hi, lo = I64(0), C.c_uint64(0)
    lib().mso_primal_value(I64(T), I64(E), I64(idx.shape[1]), _p(w), _p(idx), C.byref(hi), C.byref(lo))
    return _i128(hi, lo)


def index_build(expert_idx, E: int, Cap: int):
    """Returns (slot_idx [T,k], slot_token [E,C] with -1 padding, load [E])."""
    idx = _i32(expert_idx)
    T, k = idx.shape
    slot_idx = np.empty((T, k), np.int32)
    slot_token = np.empty((E, Cap), np.int32)
    load = np.empty(E, np.int32)
    rc = lib().mso_index_build(I64(T), I64(E), I64(k), I64(Cap), _p(idx), _p(slot_idx),
                               _p(slot_token), _p(load))
    if rc:
        raise ValueError("index_build: capacity exceeded or bad expert index")
    return slot_idx, slot_token, load


def dispatch(src: np.ndarray, slot_token) -> np.ndarray:
    """xdisp[e,s,:] = src[slot_token[e,s],:], zero rows for padding; any row dtype."""
    src = np.ascontiguousarray(src)
    st = _i32(slot_token)
    E, Cap = st.shape
    dst = np.empty((E, Cap, src.shape[1]), src.dtype)
    lib().mso_dispatch(I64(E), I64(Cap), I64(src.shape[1] * src.itemsize), _p(src), _p(st), _p(dst))
    return dst


def combine(yexp, expert_idx, slot_idx, gate_w=None) -> np.ndarray:
    """Eq. 1: Y[i] = sum_c gate_w[i,c] * yexp[e_c, slot_c]; float64 result."""
    yexp = _f64(yexp)
    E, Cap, d = yexp.shape
    idx, sl = _i32(expert_idx), _i32(slot_idx)
    T, k = idx.shape
    g = _f64(gate_w) if gate_w is not None else None
    Y = np.empty((T, d), np.float64)
    lib().mso_combine(I64(T), I64(d), I64(k), I64(Cap), _p(yexp), _p(idx), _p(sl),
                      _p(g) if g is not None else None, _p(Y))
    return Y


def combine_bwd(dY, yexp, expert_idx, slot_idx, gate_w):
    """Returns (dyexp [E,C,d], dgate_w [T,k]) in float64."""
    dY, yexp, g = _f64(dY), _f64(yexp), _f64(gate_w)
    E, Cap, d = yexp.shape
    idx, sl = _i32(expert_idx), _i32(slot_idx)
    T, k = idx.shape
    dyexp = np.empty_like(yexp)
    dg = np.empty((T, k), np.float64)
    lib().mso_combine_bwd(I64(T), I64(d), I64(E), I64(k), I64(Cap), _p(dY), _p(yexp), _p(idx),
                          _p(sl), _p(g), _p(dyexp), _p(dg))
    return dyexp, dg


def gate_bwd(H, W, dL):
    """Returns (dW [d,E], dH [T,d]) in float64."""
    H, W, dL = _f64(H), _f64(W), _f64(dL)
    T, d = H.shape
    E = W.shape[1]
    dW = np.empty((d, E), np.float64)
    dH = np.empty((T, d), np.float64)
    lib().mso_gate_bwd(I64(T), I64(d), I64(E), _p(H), _p(W), _p(dL), _p(dW), _p(dH))
    return dW, dH


def aux_loss(A, expert_idx, lam: float) -> float:
    A, idx = _f64(A), _i32(expert_idx)
    T, E = A.shape
    return float(lib().mso_aux_loss(I64(T), I64(E), I64(idx.shape[1]), C.c_double(lam), _p(A), _p(idx)))


def aux_loss_grad(expert_idx, T: int, E: int, lam: float) -> np.ndarray:
    """dL_aux/dA_ij (Eq. 9, P constant): one value per expert j, the same for every token."""
    idx = _i32(expert_idx)
    out = np.empty(E, np.float64)
    lib().mso_aux_loss_grad(I64(T), I64(E), I64(idx.shape[1]), C.c_double(lam), _p(idx), _p(out))
    return out


def gate_weights(A, expert_idx) -> np.ndarray:
    """R(x)_e = P_ie * A_ie at the assigned pairs, not renormalised (Eq. 1-2)."""
    A = np.asarray(A)
    return np.take_along_axis(A, np.asarray(expert_idx, dtype=np.int64), axis=1)


def total_score(A, expert_idx) -> float:
    """Objective of Eq. 8 in float64."""
    return float(gate_weights(_f64(A), expert_idx).sum())
