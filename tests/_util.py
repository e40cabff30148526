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


TOL = {"f32": 1e-4, "bf16": 2e-2}
