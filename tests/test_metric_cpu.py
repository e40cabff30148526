"""The error metric of the parity tests, exercised on the oracle alone (the planted mistake lives on the CPU).

Scaling the inter-chunk readout phi(Q) S_prev by 0.9 is a 10 % fault in the attention term.  With zero-mean values
and taps of unit scale the convolution branch covers it (the metric is floored at the tensor's RMS, which the
convolution sets); with zero taps, or with values drawn around 1, the same fault is far above the bf16 tolerance.
That is why the GPU parity tests carry `w0` and `vmean` variants of every mode.
"""
import numpy as np

from oracle import la_oracle as orc
from paper_2406_07368_b200 import workloads as wl
from tests._util import TOL, rel_err


def _faulty_second_half(v_mean, zero_w):
    io, B, H, d, T, W = "bf16", 1, 2, 128, 1024, 3
    q, k, v = wl.qkv(7, (B, H, T, d), d ** -0.5, io, v_mean=v_mean)
    w = wl.conv_weights(7, H, d, W)
    if zero_w:
        w = np.zeros_like(w)
    want, _ = orc.prefill_quadratic(q, k, v, w, "elu1", 0.0)
    _, half = orc.prefill_quadratic(q[:, :, :512], k[:, :, :512], v[:, :, :512], w, "elu1", 0.0)
    wrong_state = orc.State(0.9 * half.S, half.z, half.win, half.pos)
    wrong, _ = orc.prefill_quadratic(q[:, :, 512:], k[:, :, 512:], v[:, :, 512:], w, "elu1", 0.0, wrong_state)
    return rel_err(wrong, want[:, :, 512:])


def test_a_scaled_readout_hides_behind_the_convolution_and_shows_without_it():
    assert _faulty_second_half(0.0, zero_w=False) < 2 * TOL["bf16"]       # covered: the metric barely moves
    assert _faulty_second_half(0.0, zero_w=True) > 3 * TOL["bf16"]        # zero taps: o = la, the fault shows
    assert _faulty_second_half(1.0, zero_w=False) > 3 * TOL["bf16"]       # values around 1: la is of order one


def test_v_mean_shifts_only_the_values():
    q0, k0, v0 = wl.qkv(3, (1, 2, 5, 8), 1.0, "bf16")
    q1, k1, v1 = wl.qkv(3, (1, 2, 5, 8), 1.0, "bf16", v_mean=1.0)
    np.testing.assert_array_equal(q0, q1)
    np.testing.assert_array_equal(k0, k1)
    np.testing.assert_array_equal(v1, wl.round_to_bf16(v0 + np.float32(1.0)))


def test_octaves_tile_the_positions_and_see_the_fault_at_late_rows():
    from tests._util import position_octaves, rel_err_octaves
    for T in (1, 2, 3, 128, 700):
        cuts = position_octaves(T)
        assert cuts[0] == (0, 1) and cuts[-1][1] == T or T == 1
        assert all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
    # a fault confined to the last rows of a decaying signal is invisible to one RMS over the tensor, not to octaves
    T = 4096
    y = np.random.default_rng(0).standard_normal((1, 1, T, 8)) / np.sqrt(np.arange(1, T + 1))[None, None, :, None]
    x = y.copy()
    x[:, :, -256:] += 0.2 / np.sqrt(T)                  # an offset of a fifth of the late rows' own size
    assert rel_err_octaves(x, y) > 2.0 * rel_err(x, y) and rel_err_octaves(x, y) > 0.15


def test_group_octaves_pick_the_position_within_the_group():
    from tests._util import rel_err_group_octaves
    T, C = 50, 16
    y = np.ones((1, 1, T, 4))
    x = y.copy()
    assert rel_err_group_octaves(x, y, C) == 0.0
    x[0, 0, 35] *= 1.25                                  # position 3 of the third group
    assert abs(rel_err_group_octaves(x, y, C) - 0.25) < 1e-12
    # a decaying signal within each group: a fault at the group's late rows hides behind the tensor's RMS
    t = np.arange(T) % C
    y = (1.0 / (1.0 + t) ** 2)[None, None, :, None] * np.ones((1, 1, T, 4))
    x = y.copy()
    x[:, :, t >= 8] += 0.2 * y[:, :, t >= 8]
    assert rel_err(x, y) < 0.02 < 0.15 < rel_err_group_octaves(x, y, C)
