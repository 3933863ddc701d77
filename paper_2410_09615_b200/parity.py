"""Acceptance rule for a computed layer output against a float64 reference.

The output passes when both hold:
  * relative Frobenius error  ||Y - Y_ref||_F / ||Y_ref||_F <= 1e-2
  * for every element  |Y - Y_ref| <= 1e-2 * |Y_ref| + 1e-2 * rms(Y_ref)
where rms is taken over the whole reference array that is passed in.
"""
from __future__ import annotations

import numpy as np

REL_FRO_TOL = 1e-2
ELEM_REL_TOL = 1e-2
ELEM_RMS_TOL = 1e-2


def compare(y: np.ndarray, y_ref: np.ndarray) -> dict:
    y = np.asarray(y, dtype=np.float64)
    y_ref = np.asarray(y_ref, dtype=np.float64)
    assert y.shape == y_ref.shape, (y.shape, y_ref.shape)
    if y_ref.size == 0:
        return dict(ok=True, rel_fro=0.0, worst_ratio=0.0, worst_index=None, rms_ref=0.0)
    diff = np.abs(y - y_ref)
    fro_ref = float(np.sqrt(np.sum(y_ref * y_ref)))
    rel_fro = float(np.sqrt(np.sum(diff * diff))) / fro_ref if fro_ref > 0 else float(diff.max() > 0)
    rms = float(np.sqrt(np.mean(y_ref * y_ref)))
    bound = ELEM_REL_TOL * np.abs(y_ref) + ELEM_RMS_TOL * rms
    # with an all-zero reference the bound is zero and only exact zeros pass
    with np.errstate(divide="ignore", invalid="ignore"):
        ratio = np.where(bound > 0, diff / bound, np.where(diff > 0, np.inf, 0.0))
    worst = int(np.argmax(ratio))
    ok = bool(np.isfinite(y).all() and rel_fro <= REL_FRO_TOL and float(ratio.flat[worst]) <= 1.0)
    return dict(ok=ok, rel_fro=rel_fro, worst_ratio=float(ratio.flat[worst]),
                worst_index=np.unravel_index(worst, y.shape), rms_ref=rms)
