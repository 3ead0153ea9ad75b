"""Validity of a kept-token set produced in fp32 against Algorithm 1's fp64 ranking.

Step 6 keeps the k largest s^_i + m_i.  The CUDA path ranks fp32 logits, so two tokens whose
exact scores are closer than fp32 rounding may be ordered either way; everything else is
fixed.  The check below is complete: size, order, range, padding, the local window, and --
with tau the k'-th largest fp64 s^ outside the window (k' = k minus the window) -- every
token surely above tau kept, every token surely below it dropped.

The band.  A GPU logit is c32 * (a sum of r exact fp16 x fp16 products accumulated in fp32),
c32 the same positive constant for every token of the row, so it cannot change a ranking.
Whatever the order of the r additions, the accumulated sum differs from the exact dot product
by at most r u A with u = 2^-24 and A = sum_t |q_t| |k_it| over the kept dims, and the final
multiplication adds at most u |dot| <= u A.  In the exact logit's units (natural log, c =
scale / sqrt(ratio)) each logit is therefore off by at most (r + 1) u c A, and two tokens can
swap only if their exact logits differ by at most twice that.  A is bounded for the whole row
by (the sum of the r largest |q_d|) x (the largest |K| entry of the row).  Since s^ is the
exponential of the logit over a common sum, the band on the logit is a relative band on s^:
|ln s^_i - ln tau| <= delta.
"""
import math

import numpy as np

U = 2.0 ** -24


def logit_band(q_row: np.ndarray, k_abs_max: float, r: int, scale: float) -> float:
    """delta for one (sequence, head): q_row fp16 [D], k_abs_max the largest |K| entry of its rows."""
    mags = np.sort(np.abs(q_row.astype(np.float64)))[::-1]
    total = mags.sum()
    ratio = mags[:r].sum() / total if total > 0 else 1.0
    if ratio == 0.0:
        return 0.0
    c = float(np.float32(scale)) / math.sqrt(ratio)
    return 2.0 * (r + 1) * U * c * mags[:r].sum() * float(k_abs_max)


def check_kept_set(J_row: np.ndarray, s_hat: np.ndarray, S: int, k: int, l: int, delta: float, what=""):
    """J_row: int32 [>= k] from the GPU (ascending, -1 padded); s_hat: fp64 [S] from the oracle.
    Returns the number of undecided tokens: inside the band without being exact ties of tau
    (tau itself always sits at gap 0)."""
    k = min(k, S)
    window = min(l, k)
    J = J_row[:k]
    assert np.all(J_row[k:] == -1), f"{what}: padding"
    if k == 0:
        return 0
    assert J[0] >= 0 and J[-1] < S and np.all(np.diff(J) > 0), f"{what}: not ascending in [0, S)"
    kept = np.zeros(S, dtype=bool)
    kept[J] = True
    assert kept[S - window:].all(), f"{what}: a window position is missing"
    outside, want = S - window, k - window
    assert kept[:outside].sum() == want
    if want == 0 or want == outside:
        return 0
    scores = s_hat[:outside]
    tau = np.partition(scores, outside - want)[outside - want]          # the want-th largest
    with np.errstate(divide="ignore"):
        gap = np.log(scores) - math.log(tau) if tau > 0 else np.where(scores > 0, np.inf, 0.0)
    must_keep, must_drop = gap > delta, gap < -delta
    assert kept[:outside][must_keep].all(), \
        f"{what}: {int((~kept[:outside][must_keep]).sum())} tokens above the band were dropped"
    assert not kept[:outside][must_drop].any(), \
        f"{what}: {int(kept[:outside][must_drop].sum())} tokens below the band were kept"
    return int((~must_keep & ~must_drop & (gap != 0)).sum())
