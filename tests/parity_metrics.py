"""Error metrics of the GPU parity tests (plain numpy; no method arithmetic).

Per output tensor T (z, K, V, logits) the tests bound
  * the scale-relative maximum  max|T_gpu - T_ref| / max|T_ref|            (<= 1e-4 fp32, <= 2e-2 bf16 storage),
  * the worst row: max over rows (vectors along the last axis) of ||row_gpu - row_ref||_2 / ||row_ref||_2
    at the same bound, so that an error confined to a row of small norm cannot hide behind the largest
    entry of the tensor,
and they report (and loosely bound) two more figures:
  * the element-wise maximum of |D| / (|ref| + 1e-3 max|ref|).  An entry near zero carries the absolute
    error of its row (about 2^-9 of the row's typical magnitude in bf16 mode), so this figure is of
    order (row rms / max) / (1e-3 * 2^9), i.e. well above the bound of the first metric; what the
    arithmetic guarantees is 1e3 times that bound, and the tests assert a quarter of that.  The figure is the
    maximum of millions of rounding-noise samples (6.3e6 entries at config 2), an extreme-value statistic: two
    builds with the same max-norm and row errors gave 1.92 and 2.28 for the same tensor (and 1.89 / 1.55 for
    another), so a bound just above one observed value would test the noise, not the arithmetic,
  * the error by position t for [B, N, d] tensors: e(t) = max_{b,j} |D[b,t,j]| / max|ref|.  Sec. 4 argues
    that long dependency chains are damped, so e(t) must not grow along the sequence: the maximum over the
    last quarter of the positions may not exceed ten times the maximum over the first quarter (or a floor
    of a twentieth of the bound, whichever is larger).
A line per tensor is appended to the file named by the environment variable RT_PARITY_REPORT, if set.
"""
import json
import os

import numpy as np


def max_norm_err(got, ref):
    return float(np.abs(got - ref).max() / np.abs(ref).max())


def row_rel_err(got, ref):
    num = np.sqrt(((got - ref) ** 2).sum(axis=-1))
    den = np.sqrt((ref ** 2).sum(axis=-1))
    floor = 1e-6 * float(den.max()) if den.size else 0.0
    return float((num / np.maximum(den, floor)).max())


def elementwise_err(got, ref):
    m = float(np.abs(ref).max())
    return float((np.abs(got - ref) / (np.abs(ref) + 1e-3 * m)).max())


def position_curve(got, ref):
    """e(t) for tensors laid out [B, N, ...]; None otherwise."""
    if got.ndim < 3:
        return None
    d = np.abs(got - ref)
    return d.reshape(d.shape[0], d.shape[1], -1).max(axis=(0, 2)) / float(np.abs(ref).max())


def check_tensor(what, name, got, ref, tol, curve=True):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, f"{what}: {name} shape {got.shape} != {ref.shape}"
    assert np.isfinite(got).all(), f"{what}: non-finite {name}"
    e_max, e_row, e_el = max_norm_err(got, ref), row_rel_err(got, ref), elementwise_err(got, ref)
    rec = {"case": what, "tensor": name, "max_norm": e_max, "row_rel_l2": e_row, "elementwise": e_el, "tol": tol}
    c = position_curve(got, ref) if curve else None
    if c is not None and c.size >= 64:
        q = c.size // 4
        early, late = float(c[:q].max()), float(c[-q:].max())
        rec["by_position_quartile_max"] = [float(c[i * q:(i + 1) * q].max()) for i in range(4)]
        assert late <= max(10.0 * early, tol / 20.0), f"{what}: {name} error grows along the sequence: {rec}"
    path = os.environ.get("RT_PARITY_REPORT")
    if path:
        with open(path, "a") as f:
            f.write(json.dumps(rec) + "\n")
    assert e_max <= tol, f"{what}: {name} max-norm error {e_max:.3e} > {tol}"
    assert e_row <= tol, f"{what}: {name} worst-row relative error {e_row:.3e} > {tol}"
    assert e_el <= 250.0 * tol, f"{what}: {name} element-wise error {e_el:.3e} > {250.0 * tol}"
    return rec
