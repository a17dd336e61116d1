"""Shared helpers of the GPU parity tests: the tolerance gate between the CUDA path and the CPU
checker.

Attention and row-softmax results are compared element by element.  The bar is max-abs 1e-2 and
mean-abs 1e-3 in fp32 units.  The CUDA path forms scores in fp32 (tensor cores) while the
checker uses double, so a quantity sitting on a decision boundary can legitimately land on the
other side; the checker reports, per row,
  * ``row_allow``  -- a bound on the output change if the element roundings that lie within
    2^-16 (relative) of a HiF8 rounding boundary had gone the other way, and
  * ``row_margin`` -- the distance of the row's max / restart / delta decisions to their
    boundaries;
rows are gated at 1e-2 + row_allow, rows with a decision margin below 2^-16 at 5e-2 + row_allow,
and such rows must stay a small fraction of all rows.  Both arrays are pinned by hand-worked cases
in test_oracle_attention.py.  Beside the gate the raw statistics are asserted: at least 99.5 % of
the rows meet the plain 1e-2 bound with no allowance at all, and a row that needs its allowance
consumes no more than the allowance itself.
"""
from __future__ import annotations

import numpy as np

EPS_REL = 2.0 ** -16
MAX_ABS = 1e-2
MEAN_ABS = 1e-3


def gate_attention(got: np.ndarray, ref, *, max_near_frac: float = 0.01, what: str = ""):
    """got: [n_sel, bq, D] float; ref: oracle.AttentionResult for the same tiles."""
    got = np.asarray(got, dtype=np.float64).reshape(ref.out.shape)
    err = np.abs(got - ref.out)
    near = ref.row_margin < EPS_REL
    row_err = err.max(axis=-1)
    tol = MAX_ABS + ref.row_allow + np.where(near, 4e-2, 0.0)
    bad = row_err > tol
    plain_ok = row_err <= MAX_ABS                   # rows that need neither allowance nor margin slack
    info = dict(max_abs=float(err.max()), mean_abs=float(err.mean()), near_frac=float(near.mean()),
                plain_frac=float(plain_ok.mean()), worst_excess=float((row_err - tol).max()),
                allowance_used=float(np.where(~plain_ok & ~near, row_err - MAX_ABS, 0.0).max()))
    assert not bad.any(), f"{what}: {int(bad.sum())} rows over tolerance: {info}"
    assert err.mean() <= MEAN_ABS, f"{what}: mean-abs too large: {info}"
    assert plain_ok.mean() >= 0.995, f"{what}: too many rows need an allowance: {info}"
    if near.size >= 128:
        assert near.mean() <= max_near_frac, f"{what}: too many near-boundary rows: {info}"
    return info


def gate_softmax_rows(got: np.ndarray, probs: np.ndarray, margin: np.ndarray, allow: np.ndarray,
                      what: str = ""):
    got = np.asarray(got, dtype=np.float64)
    err = np.abs(got - probs)
    near = margin < EPS_REL
    tol = MAX_ABS + allow + np.where(near, 4e-2, 0.0)[:, None]
    plain_ok = err.max(axis=1) <= MAX_ABS
    info = dict(max_abs=float(err.max()), mean_abs=float(err.mean()), near_rows=int(near.sum()),
                plain_frac=float(plain_ok.mean()))
    assert np.all(err <= tol), f"{what}: elements over tolerance: {info}"
    assert plain_ok.mean() >= 0.995, f"{what}: too many rows need an allowance: {info}"
    if near.size >= 128:
        assert near.mean() <= 0.01, f"{what}: too many near-boundary rows: {info}"
    assert err.mean() <= MEAN_ABS, f"{what}: {info}"
    assert np.abs(got.sum(axis=1) - 1.0).max() <= 1e-4, f"{what}: rows do not sum to one"
    return info
