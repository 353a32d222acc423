"""Comparison protocol between a device result (given as numpy arrays) and the CPU oracle.

Test infrastructure only.  It never imports the CUDA binding: callers hand it arrays.  The
protocol keeps channel-pick differences and value errors apart:

1. picks: for every token, the symmetric difference between the device's channel set and the
   oracle's may contain only channels whose oracle gate value lies within ``band`` (absolute,
   pre-SiLU) of the oracle's K-th largest gate value of that token;
2. values: out / gate / up values are compared with the oracle evaluated on the DEVICE's channel
   sets (``forward_given_idx``), so a legitimate near-tie pick does not show up as a value error;
3. backward: both sides consume the same saved tensors and the same upstream gradient.

Tolerance: max-abs error <= rel * max|reference| per tensor, rel = 1e-2 for bf16 storage and
1e-4 for fp32 storage.
"""
from __future__ import annotations

import numpy as np

from . import moc_oracle as orc

REL_TOL = {"bf16": 1e-2, "f32": 1e-4}
PICK_BAND = 1e-3


def max_err(got: np.ndarray, ref: np.ndarray):
    """(max abs error, max |ref|)"""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    if got.shape != ref.shape:
        raise AssertionError(f"shape mismatch {got.shape} vs {ref.shape}")
    if got.size == 0:
        return 0.0, 0.0
    if not np.all(np.isfinite(got)):
        return float("inf"), float(np.abs(ref).max())
    return float(np.abs(got - ref).max()), float(np.abs(ref).max())


def assert_close(got, ref, dtype: str, what: str, rel: float | None = None):
    rel = REL_TOL[dtype] if rel is None else rel
    err, scale = max_err(got, ref)
    bound = rel * scale
    if not err <= bound + 1e-30:
        raise AssertionError(f"{what}: max-abs error {err:.3e} exceeds {rel:g} * max|ref| = {bound:.3e}")
    return err, scale


def check_index_sets(idx: np.ndarray, F: int):
    """Structural validity: K distinct ascending channels in [0, F) per token."""
    idx = np.asarray(idx).astype(np.int64)
    if idx.size == 0:
        return
    if idx.min() < 0 or idx.max() >= F:
        raise AssertionError("channel index out of range")
    if idx.shape[1] > 1 and not np.all(np.diff(idx, axis=1) > 0):
        raise AssertionError("channel indices not strictly ascending within a token")


def check_picks(idx_dev: np.ndarray, g_oracle: np.ndarray, K: int, band: float = PICK_BAND):
    """Rule 1.  Returns the number of tokens whose set differs from the oracle's (all inside the band)."""
    idx_ref = orc.topk(g_oracle, K)
    idx_dev = np.asarray(idx_dev).astype(np.int64)
    T, F = g_oracle.shape
    check_index_sets(idx_dev, F)
    differing = 0
    key = np.where(np.isnan(g_oracle), -np.inf, g_oracle)
    for t in range(T):
        a, b = set(idx_dev[t].tolist()), set(idx_ref[t].tolist())
        if a == b:
            continue
        differing += 1
        tau = np.min(key[t, idx_ref[t]])
        for j in a ^ b:
            if not abs(key[t, j] - tau) <= band:
                raise AssertionError(
                    f"token {t}: channel {j} (g={key[t, j]!r}) differs from the oracle's pick outside the "
                    f"{band:g} band around tau={tau!r}")
    return differing


def check_forward(dev: dict, x, w_gate, w_up, w_down, K: int, F: int, dtype: str, g_oracle=None):
    """dev: dict(out, idx, gval, uval) as float64/int arrays (gval/uval may be None).  Returns a report dict."""
    rep = {}
    if g_oracle is None:
        g_oracle = orc.forward(x, w_gate, w_up, w_down, K, F=F, want_g=True)["g"]
    rep["tokens_with_band_picks"] = check_picks(dev["idx"], g_oracle, K)
    ref = orc.forward_given_idx(x, w_gate, w_up, w_down, np.asarray(dev["idx"], dtype=np.int32), F=F)
    rep["out"] = assert_close(dev["out"], ref["out"], dtype, "out")
    if dev.get("gval") is not None:
        rep["gval"] = assert_close(dev["gval"], ref["gval"], dtype, "topk_gate")
    if dev.get("uval") is not None:
        rep["uval"] = assert_close(dev["uval"], ref["uval"], dtype, "topk_up")
    return rep


def check_backward(dev: dict, x, w_gate, w_up, w_down, idx, gval, uval, grad_out, F: int, dtype: str):
    """dev: dict(grad_x, grad_w_gate, grad_w_up, grad_w_down), entries may be None.  Saved tensors are the
    ones the device consumed (already widened to float64)."""
    want = tuple(n for n in ("x", "w_gate", "w_up", "w_down") if dev.get("grad_" + n) is not None)
    ref = orc.backward(x, w_gate, w_up, w_down, np.asarray(idx, dtype=np.int32), gval, uval, grad_out, F=F,
                       want=want)
    rep = {}
    for n in want:
        got = np.asarray(dev["grad_" + n], dtype=np.float64)
        if n != "x" and got.shape[0] > F:
            if np.any(got[F:] != 0.0):
                raise AssertionError(f"grad_{n}: padding rows are not zero")
            got = got[:F]
        rep["grad_" + n] = assert_close(got, ref["grad_" + n], dtype, "grad_" + n)
    return rep


def check_picks_grouped(idx_dev: np.ndarray, g_oracle: np.ndarray, group: int = 8, keep: int = 2,
                        band: float = PICK_BAND):
    """Rule 1 for the grouped (a:b) mask: per token and group, the device's channels may differ from the oracle's
    only by channels whose oracle gate value lies within ``band`` of that group's keep-th largest value.
    Returns the number of groups whose set differs."""
    idx_ref = orc.topk_grouped(g_oracle, group, keep)
    idx_dev = np.asarray(idx_dev).astype(np.int64)
    T, F = g_oracle.shape
    check_index_sets(idx_dev, F)
    groups = F // group
    if idx_dev.shape != (T, groups * keep):
        raise AssertionError(f"grouped index shape {idx_dev.shape}")
    if not np.array_equal(idx_dev // group, np.repeat(np.arange(groups), keep)[None, :].repeat(T, axis=0)):
        raise AssertionError("not exactly `keep` channels in every group")
    key = np.where(np.isnan(g_oracle), -np.inf, g_oracle)
    differing = 0
    diff_rows, diff_cols = np.nonzero(idx_dev != idx_ref)
    for t, c in zip(diff_rows.tolist(), diff_cols.tolist()):
        q = c // keep
        vals = np.sort(key[t, q * group:(q + 1) * group])[::-1]
        tau = vals[keep - 1]
        a = set(idx_dev[t, q * keep:(q + 1) * keep].tolist())
        b = set(idx_ref[t, q * keep:(q + 1) * keep].tolist())
        for j in a ^ b:
            if abs(key[t, j] - tau) > band:
                raise AssertionError(f"token {t} group {q}: channel {j} (g={key[t, j]:.6g}) differs outside the band "
                                     f"around {tau:.6g}")
        differing += 1
    return differing


def check_decode(out, x, w_gate, w_up, w_down, K: int, dtype: str, what: str = "decode"):
    """A decode result (no indices come back) against the oracle's own picks.  Where a token's margin between its K-th
    and (K+1)-th gate value is below 1e-4 (inside the exclusion band) the swapped pick is accepted as well; every other
    token must match within the tolerance.  Arrays are float64; weights hold the logical channels only."""
    full = orc.forward(x, w_gate, w_up, w_down, K, want_g=True)
    F = w_gate.shape[0]
    scale = np.abs(full["out"]).max()
    tol = REL_TOL[dtype] * scale
    for t in range(x.shape[0]):
        err = np.abs(out[t] - full["out"][t]).max()
        if err <= tol:
            continue
        g = full["g"][t]
        order = np.lexsort((np.arange(F), -g))
        if not (K < F and g[order[K - 1]] - g[order[K]] <= 1e-4):
            raise AssertionError(f"{what}: token {t} error {err:.3e} > {tol:.3e}")
        alt = np.sort(np.concatenate([order[: K - 1], order[K: K + 1]])).astype(np.int32)[None]
        ref = orc.forward_given_idx(x[t: t + 1], w_gate, w_up, w_down, alt)["out"][0]
        if not np.abs(out[t] - ref).max() <= tol:
            raise AssertionError(f"{what}: token {t} matches neither pick")
