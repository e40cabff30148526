"""Helpers shared by the tests: the error metric and small conversions."""
import numpy as np


def rel_err(x, y) -> float:
    """max_i |x_i - y_i| / max(|y_i|, rms(y)) over one tensor (y is the expected value).

    The floor at the tensor's RMS keeps elements that pass through zero from
    dominating; everything else is a plain elementwise relative error.
    """
    x = np.asarray(x, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    assert x.shape == y.shape, (x.shape, y.shape)
    if y.size == 0:
        return 0.0
    tau = float(np.sqrt(np.mean(y * y)))
    if tau == 0.0:
        return float(np.max(np.abs(x - y)))
    return float(np.max(np.abs(x - y) / np.maximum(np.abs(y), tau)))


def position_octaves(T: int):
    """[0, 1), [1, 2), [2, 4), [4, 8), ... up to T: ranges of positions within which the attention term of a fresh
    sequence keeps its scale to within a factor of about sqrt(2)."""
    out, lo = [(0, 1)], 1
    while lo < T:
        out.append((lo, min(2 * lo, T)))
        lo *= 2
    return out


def rel_err_octaves(x, y, axis: int = 2) -> float:
    """rel_err taken octave by octave along the position axis, each octave against its own RMS; the largest.

    With zero taps and zero-mean values the output is a running weighted mean of the values: of the values' own
    size in the first rows and about 1/sqrt(i) of it at row i.  One RMS over the whole tensor is then several
    times smaller than the early rows and several times larger than the late ones, so it is neither a fair floor
    for the former nor a strict one for the latter; an octave of positions shares one scale.
    """
    x, y = np.asarray(x), np.asarray(y)
    worst = 0.0
    for lo, hi in position_octaves(y.shape[axis]):
        sl = [slice(None)] * y.ndim
        sl[axis] = slice(lo, hi)
        worst = max(worst, rel_err(x[tuple(sl)], y[tuple(sl)]))
    return worst


def rel_err_group_octaves(x, y, group: int, axis: int = 2) -> float:
    """rel_err per octave of the position WITHIN a group of `group` tokens (all groups together), the largest.

    The local branch of the three-branch block is a softmax mean over the tokens of the group so far, so with zero
    taps and zero-mean values the output's scale follows the position in the group the way rel_err_octaves
    describes for the position in a fresh sequence.
    """
    x, y = np.asarray(x), np.asarray(y)
    t = np.arange(y.shape[axis]) % group
    worst = 0.0
    for lo, hi in position_octaves(group):
        pick = np.nonzero((t >= lo) & (t < hi))[0]
        worst = max(worst, rel_err(np.take(x, pick, axis=axis), np.take(y, pick, axis=axis)))
    return worst


TOL = {"f32": 1e-4, "bf16": 2e-2}
