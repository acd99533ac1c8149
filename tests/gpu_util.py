"""Helpers shared by the GPU parity tests (no routing arithmetic here)."""
import numpy as np
import torch


def f64(t: torch.Tensor) -> np.ndarray:
    """Exact float64 image of an fp32 / bf16 tensor."""
    return t.detach().to("cpu").to(torch.float64).numpy()


def np32(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float32).numpy()


def raw16(t: torch.Tensor) -> np.ndarray:
    """Bit pattern of a bf16 tensor as uint16 (for bit-exact row comparisons)."""
    return t.detach().to("cpu").view(torch.int16).numpy().view(np.uint16)


def assert_rel(got, ref, tol, what=""):
    """For outputs whose terms all have one sign (no cancellation): per row
    max_i |d_i| <= tol * max_i |ref_i|, and elementwise |d| <= tol*|ref| wherever
    |ref| >= 1e-4 * rowmax."""
    got = np.asarray(got, dtype=np.float64).reshape(-1, got.shape[-1])
    ref = np.asarray(ref, dtype=np.float64).reshape(-1, ref.shape[-1])
    rowmax = np.abs(ref).max(axis=1, keepdims=True)
    d = np.abs(got - ref)
    assert (d <= tol * rowmax + 1e-300).all(), f"{what}: row-relative error {np.max(d / (rowmax + 1e-300)):.3e} > {tol}"
    big = (np.abs(ref) >= 1e-4 * rowmax) & (rowmax > 0)
    rel = d[big] / np.abs(ref[big])
    assert rel.size == 0 or rel.max() <= tol, f"{what}: elementwise relative error {rel.max():.3e} > {tol}"


def assert_sum_close(got, ref, mag, tol, what=""):
    """For outputs that are sums of signed products: |got - ref| <= tol * mag elementwise, where mag is
    the same sum taken over absolute values (the magnitude the rounding errors scale with).  Entries
    whose magnitude is zero must be exactly zero."""
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    mag = np.asarray(mag, dtype=np.float64)
    d = np.abs(got - ref)
    bad = d > tol * mag
    assert not bad.any(), f"{what}: {bad.sum()} entries off, worst {np.max(d / (mag + 1e-300)):.3e} > {tol}"


def assert_row_rel(got, ref, tol, what=""):
    """Row-relative bar for sums of signed products: per row max_i |d_i| <= tol * max_i |ref_i|.  Returns the
    worst ratio seen, so that callers can report it."""
    got = np.asarray(got, dtype=np.float64).reshape(-1, got.shape[-1])
    ref = np.asarray(ref, dtype=np.float64).reshape(-1, ref.shape[-1])
    rowmax = np.abs(ref).max(axis=1)
    d = np.abs(got - ref).max(axis=1)
    worst = float(np.max(d / (rowmax + 1e-300)))
    assert (d <= tol * rowmax + 1e-300).all(), f"{what}: row-relative error {worst:.3e} > {tol}"
    return worst


def assert_rounded_sum_close(got, ref, mag, tol_acc, what=""):
    """For outputs that are sums of signed products accumulated in fp32 and rounded ONCE to bf16:
    |got - ref| <= 2^-8 |ref| + tol_acc * mag elementwise (one bf16 rounding of the result plus the
    accumulation error, which scales with the sum of the absolute terms `mag`).  A dropped tile, expert
    column or half of a split operand is far outside this bar."""
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    mag = np.asarray(mag, dtype=np.float64)
    d = np.abs(got - ref)
    bar = 2.0 ** -8 * np.abs(ref) + tol_acc * mag
    bad = d > bar
    assert not bad.any(), f"{what}: {bad.sum()} entries off, worst {np.max(d / (bar + 1e-300)):.3f} x the bar"


def float_keys(scores32: np.ndarray) -> np.ndarray:
    """The keys the library documents for score_mode 0 (include/maxscore.h), computed by the oracle."""
    import oracle
    return oracle.keys_from_scores_hashed(np.asarray(scores32, dtype=np.float32).astype(np.float64))
