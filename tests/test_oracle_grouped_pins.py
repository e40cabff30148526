"""Pins of the oracle's three-branch block (Sec. 4.1: grouped linear attention between groups, softmax attention
inside a group, masked depthwise convolution, alpha).  None of them re-types the oracle's formula: a hand-worked
example, library softmax attention, already pinned oracle functions reached by another route, scalar brute force."""
import json
import math
import os
from fractions import Fraction

import numpy as np
import torch

from oracle import la_oracle as orc

HERE = os.path.dirname(os.path.abspath(__file__))
RNG = np.random.default_rng(11)


def rand(B, H, T, d, W):
    q, k, v = (RNG.standard_normal((B, H, T, d)) for _ in range(3))
    return q, k, v, RNG.standard_normal((H, d, W)) * W ** -0.5


def sdpa(q, k, v, scale):
    """Library causal softmax attention (float64)."""
    return torch.nn.functional.scaled_dot_product_attention(torch.tensor(q), torch.tensor(k), torch.tensor(v),
                                                            is_causal=True, scale=scale).numpy()


def test_hand_worked_two_group_example():
    g = json.load(open(os.path.join(HERE, "golden", "hand_example_grouped.json")))
    s, e = g["setup"], g["expected"]
    sh = (1, 1, 4, 1)
    q = np.array(s["q"], dtype=np.float64).reshape(sh)
    k = (np.array(s["k_over_ln2"], dtype=np.float64) * math.log(2.0)).reshape(sh)
    v = np.array(s["v"], dtype=np.float64).reshape(sh)
    w = np.array(s["w"], dtype=np.float64).reshape(1, 1, 2)
    o, st = orc.prefill_grouped_block(q, k, v, w, s["phi"], s["eps"], s["group"], s["alpha"], s["scale"])
    want = [float(Fraction(a, b)) for a, b in e["o_fractions"]]
    np.testing.assert_allclose(o.reshape(-1), want, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(st.S.reshape(-1), [e["S_over_ln2"] * math.log(2.0)], rtol=1e-13)
    np.testing.assert_allclose(st.z.reshape(-1), [e["z_over_ln2"] * math.log(2.0)], rtol=1e-13)
    assert st.win.reshape(-1).tolist() == e["win"] and st.pos.tolist() == [e["pos"]]


def test_one_group_covering_the_sequence_is_plain_causal_softmax_plus_convolution():
    B, H, T, d, W = 2, 2, 37, 8, 3
    q, k, v, w = rand(B, H, T, d, W)
    for group in (T, T + 5, 1000):
        for alpha in (0.0, 0.3, 1.0):                      # no earlier group: alpha has nothing to weigh
            o, _ = orc.prefill_grouped_block(q, k, v, w, "elu1", 0.0, group, alpha, d ** -0.5)
            want = sdpa(q, k, v, d ** -0.5) + orc.causal_dwconv(v, w, np.zeros((B, H, W - 1, d)))
            np.testing.assert_allclose(o, want, rtol=1e-11, atol=1e-12)


def test_alpha_zero_is_softmax_attention_group_by_group_plus_convolution():
    B, H, T, d, W, C = 1, 3, 29, 4, 4, 8
    q, k, v, w = rand(B, H, T, d, W)
    o, _ = orc.prefill_grouped_block(q, k, v, w, "relu", 1e-6, C, 0.0, 0.5)
    want = orc.causal_dwconv(v, w, np.zeros((B, H, W - 1, d)))
    for lo in range(0, T, C):
        sl = slice(lo, min(lo + C, T))
        want[:, :, sl] += sdpa(q[:, :, sl], k[:, :, sl], v[:, :, sl], 0.5)
    np.testing.assert_allclose(o, want, rtol=1e-11, atol=1e-12)


def test_global_branch_is_a_readout_of_the_state_before_the_group():
    """alpha * glob = (block at alpha) - (block at alpha = 0).  The same readout by another route: the recurrence's
    decode step (pinned elsewhere) with a key that ReLU maps to zero leaves the state as it is, so its attention
    term is phi(q)^T S / (phi(q) . z + eps) for the state of the groups before."""
    B, H, T, d, W, C, eps, alpha = 1, 2, 23, 6, 1, 5, 1e-3, 0.8
    q, k, v, _ = rand(B, H, T, d, W)
    w = np.zeros((H, d, W))
    o1, _ = orc.prefill_grouped_block(q, k, v, w, "relu", eps, C, alpha, 0.4)
    o0, _ = orc.prefill_grouped_block(q, k, v, w, "relu", eps, C, 0.0, 0.4)
    for i in range(T):
        g0 = (i // C) * C
        if g0 == 0:
            want = np.zeros((B, H, d))
        else:
            _, st = orc.prefill_quadratic(q[:, :, :g0], k[:, :, :g0], v[:, :, :g0], w, "relu", eps)
            null_k = -np.ones((B, H, d))
            want, _ = orc.decode_step(q[:, :, i], null_k, np.zeros((B, H, d)), w, "relu", eps, st)
        np.testing.assert_allclose(o1[:, :, i] - o0[:, :, i], alpha * want, rtol=1e-10, atol=1e-12)


def test_scalar_brute_force():
    B, H, T, d, W, C, eps, alpha, scale = 1, 1, 7, 2, 2, 3, 0.0, 0.6, 0.7
    q, k, v, w = rand(B, H, T, d, W)
    o, _ = orc.prefill_grouped_block(q, k, v, w, "elu1", eps, C, alpha, scale)
    f = lambda x: x + 1.0 if x > 0 else math.exp(x)
    for i in range(T):
        g0 = (i // C) * C
        for c in range(d):
            num = den = 0.0
            for j in range(g0):                                  # earlier groups only
                a = sum(f(q[0, 0, i, e]) * f(k[0, 0, j, e]) for e in range(d))
                num += a * v[0, 0, j, c]
                den += a
            glob = num / den if g0 > 0 else 0.0
            logits = [scale * sum(q[0, 0, i, e] * k[0, 0, j, e] for e in range(d)) for j in range(g0, i + 1)]
            ws = [math.exp(x) for x in logits]
            loc = sum(p * v[0, 0, j, c] for p, j in zip(ws, range(g0, i + 1))) / sum(ws)
            conv = sum(w[0, c, t] * v[0, 0, i - t, c] for t in range(W) if i - t >= 0)
            assert abs(o[0, 0, i, c] - (alpha * glob + loc + conv)) < 1e-12


def test_groups_of_one_token():
    """Every token its own group: the local branch returns v_i, the global branch is linear attention over all
    strictly earlier tokens."""
    B, H, T, d, W = 1, 2, 9, 3, 1
    q, k, v, _ = rand(B, H, T, d, W)
    w = np.zeros((H, d, W))
    o, _ = orc.prefill_grouped_block(q, k, v, w, "elu1", 0.0, 1, 1.0, 1.0)
    full, _ = orc.prefill_quadratic(q, k, v, w, "elu1", 0.0)
    fq, fk = orc.phi(q, "elu1"), orc.phi(k, "elu1")
    a_ii = np.einsum("bhia,bhia->bhi", fq, fk)
    den_incl = np.einsum("bhia,bhja->bhij", fq, fk)
    den_incl = np.tril(den_incl).sum(-1)
    # inclusive attention = (exclusive numerator + a_ii v_i) / (exclusive denominator + a_ii)
    excl = (full * den_incl[..., None] - a_ii[..., None] * v) / np.where(den_incl - a_ii > 0, den_incl - a_ii, 1.0)[..., None]
    excl[:, :, 0] = 0.0
    np.testing.assert_allclose(o, v + excl, rtol=1e-9, atol=1e-11)


def test_causal_under_perturbation_and_group_isolation():
    B, H, T, d, W, C = 1, 2, 26, 4, 3, 8
    q, k, v, w = rand(B, H, T, d, W)
    o, _ = orc.prefill_grouped_block(q, k, v, w, "elu1", 0.0, C, 0.5, 0.5)
    j = 13
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    q2[:, :, j] += 1.0
    k2[:, :, j] -= 2.0
    v2[:, :, j] *= 3.0
    o2, _ = orc.prefill_grouped_block(q2, k2, v2, w, "elu1", 0.0, C, 0.5, 0.5)
    assert np.array_equal(o[:, :, :j], o2[:, :, :j]) and not np.array_equal(o[:, :, j], o2[:, :, j])
    assert not np.allclose(o[:, :, 16:], o2[:, :, 16:])         # later groups see token 13 through the group sums


def test_continuation_at_a_group_boundary_and_state_totals():
    B, H, T, d, W, C = 2, 2, 31, 4, 3, 6
    q, k, v, w = rand(B, H, T, d, W)
    o, st = orc.prefill_grouped_block(q, k, v, w, "relu", 1e-6, C, 0.7, 0.5)
    cut = 3 * C
    o1, s1 = orc.prefill_grouped_block(q[:, :, :cut], k[:, :, :cut], v[:, :, :cut], w, "relu", 1e-6, C, 0.7, 0.5)
    o2, s2 = orc.prefill_grouped_block(q[:, :, cut:], k[:, :, cut:], v[:, :, cut:], w, "relu", 1e-6, C, 0.7, 0.5, s1)
    np.testing.assert_allclose(np.concatenate([o1, o2], axis=2), o, rtol=1e-12, atol=1e-13)
    _, ref = orc.prefill_quadratic(q, k, v, w, "relu", 1e-6)     # the state is the plain totals
    for a, b in ((st.S, ref.S), (st.z, ref.z), (s2.S, ref.S), (s2.z, ref.z)):
        np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)
    assert np.array_equal(st.win, ref.win) and np.array_equal(s2.win, ref.win) and st.pos.tolist() == [T] * B
    try:
        orc.prefill_grouped_block(q[:, :, :4], k[:, :, :4], v[:, :, :4], w, "relu", 1e-6, C, 0.7, 0.5,
                                  orc.State(s1.S, s1.z, s1.win, s1.pos + 1))
        raise AssertionError("a state that does not end at a group boundary must be refused")
    except ValueError:
        pass


def test_planted_mistakes_fail_the_hand_example():
    """The mistakes live here, on the CPU: a global branch that includes the token's own group, and a local branch
    without the causal mask, both miss the hand-worked values."""
    g = json.load(open(os.path.join(HERE, "golden", "hand_example_grouped.json")))
    s = g["setup"]
    ln2 = math.log(2.0)
    q, m, v = s["q"], s["k_over_ln2"], s["v"]
    want = [float(Fraction(a, b)) for a, b in g["expected"]["o_fractions"]]

    def block(inclusive_global, causal_local):
        out = []
        for i in range(4):
            g0 = (i // 2) * 2
            hi = g0 + 2 if inclusive_global else g0
            num = sum(m[j] * v[j] for j in range(hi))
            den = sum(m[j] for j in range(hi))
            glob = num / den if den else 0.0
            js = range(g0, i + 1) if causal_local else range(g0, g0 + 2)
            ws = [2.0 ** (q[i] * m[j]) for j in js]
            loc = sum(p * v[j] for p, j in zip(ws, js)) / sum(ws)
            conv = 0.5 * v[i] - (v[i - 1] if i else 0.0)
            out.append(0.5 * glob + loc + conv)
        return out
    np.testing.assert_allclose(block(False, True), want, rtol=1e-13)
    assert not np.allclose(block(True, True), want) and not np.allclose(block(False, False), want)
    _ = ln2
