"""Pins for the float64 oracle: each test fixes it to something other than itself."""
import json
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import la_oracle as orc
from paper_2406_07368_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rand(seed, shape, scale=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * scale


# ---------------------------------------------------------------- hand-worked values
def test_hand_example_prefill():
    g = json.load(open(os.path.join(GOLD, "hand_example_relu.json")))
    q, k, v = (np.array(g[n], dtype=np.float64)[None, None] for n in "qkv")
    w = np.array(g["w"])[None]
    for form in ("quadratic", "recurrent", "chunked"):
        if form == "quadratic":
            o, st = orc.prefill_quadratic(q, k, v, w, g["phi"], g["eps"])
        elif form == "recurrent":
            o, st = orc.prefill_recurrent(q, k, v, w, g["phi"], g["eps"])
        else:
            o, st = orc.prefill_chunked(q, k, v, w, g["phi"], g["eps"], 2)
        np.testing.assert_allclose(o[0, 0], np.array(g["o"]), rtol=0, atol=1e-14)
        np.testing.assert_allclose(st.S[0, 0], np.array(g["S"]), rtol=0, atol=1e-14)
        np.testing.assert_allclose(st.z[0, 0], np.array(g["z"]), rtol=0, atol=1e-14)
        np.testing.assert_array_equal(st.win[0, 0], np.array(g["win"], dtype=np.float64))
        assert st.pos[0] == g["pos"]
    # with zero taps the output is the attention term alone
    o, _ = orc.prefill_quadratic(q, k, v, np.zeros_like(w), g["phi"], g["eps"])
    np.testing.assert_allclose(o[0, 0], np.array(g["la"]), rtol=0, atol=1e-14)


def test_hand_example_tree_and_commit():
    g0 = json.load(open(os.path.join(GOLD, "hand_example_relu.json")))
    g = json.load(open(os.path.join(GOLD, "hand_example_tree.json")))
    q0, k0, v0 = (np.array(g0[n], dtype=np.float64)[None, None] for n in "qkv")
    w = np.array(g0["w"])[None]
    _, st = orc.prefill_quadratic(q0, k0, v0, w, "relu", 0.0)
    q, k, v = (np.array(g[n], dtype=np.float64)[None, None] for n in "qkv")
    parent = np.array([g["parent"]], dtype=np.int32)
    before = st.copy()
    o = orc.verify_tree(q, k, v, parent, w, "relu", 0.0, st)
    np.testing.assert_allclose(o[0, 0], np.array(g["o"]), rtol=0, atol=1e-14)
    for a, b in zip((st.S, st.z, st.win, st.pos), (before.S, before.z, before.win, before.pos)):
        np.testing.assert_array_equal(a, b)
    new, path, clen = orc.commit(k, v, parent, np.array([g["accept_node"]]), "relu", st, max_depth=4)
    assert clen[0] == g["commit_len"]
    assert list(path[0]) == g["path"] + [-1] * (4 - len(g["path"]))
    np.testing.assert_allclose(new.S[0, 0], np.array(g["S_after"]), atol=1e-14)
    np.testing.assert_allclose(new.z[0, 0], np.array(g["z_after"]), atol=1e-14)
    np.testing.assert_array_equal(new.win[0, 0], np.array(g["win_after"], dtype=np.float64))
    assert new.pos[0] == g["pos_after"]


# ---------------------------------------------------------------- closed forms
def test_geometric_series_closed_form():
    """d = 1, ReLU, q = 1, k_j = r^j, v_j = s^j: both sums are geometric series."""
    r, s, T = 0.9, 1.1, 40
    j = np.arange(T)
    q = np.ones((1, 1, T, 1))
    k = (r ** j).reshape(1, 1, T, 1)
    v = (s ** j).reshape(1, 1, T, 1)
    w = np.zeros((1, 1, 1))
    num = ((r * s) ** (j + 1) - 1) / (r * s - 1)
    den = (r ** (j + 1) - 1) / (r - 1)
    for fn in (orc.prefill_quadratic, orc.prefill_recurrent):
        o, st = fn(q, k, v, w, "relu", 0.0)
        np.testing.assert_allclose(o[0, 0, :, 0], num / den, rtol=1e-13)
        np.testing.assert_allclose(st.S[0, 0, 0, 0], num[-1], rtol=1e-13)
        np.testing.assert_allclose(st.z[0, 0, 0], den[-1], rtol=1e-13)
    o, _ = orc.prefill_chunked(q, k, v, w, "relu", 0.0, 7)
    np.testing.assert_allclose(o[0, 0, :, 0], num / den, rtol=1e-13)
    # eps enters the denominator additively
    o, _ = orc.prefill_quadratic(q, k, v, w, "relu", 0.5)
    np.testing.assert_allclose(o[0, 0, :, 0], num / (den + 0.5), rtol=1e-13)


def test_elu1_values():
    """phi(x) = x + 1 for x > 0, exp(x) otherwise: check against math.exp and continuity at 0."""
    import math
    xs = [-3.0, -1.0, -1e-9, 0.0, 1e-9, 0.5, 2.0]
    got = orc.phi(np.array(xs), "elu1")
    want = [math.exp(-3.0), math.exp(-1.0), math.exp(-1e-9), 1.0, 1.0 + 1e-9, 1.5, 3.0]
    np.testing.assert_allclose(got, want, rtol=1e-15)
    np.testing.assert_array_equal(orc.phi(np.array([-2.0, 0.0, 3.0]), "relu"), [0.0, 0.0, 3.0])
    assert np.all(orc.phi(_rand(0, (1000,)) * 5, "elu1") > 0)


def test_single_token_returns_v():
    """T = 1, eps = 0: the only weight cancels, la_0 = v_0, so o_0 = v_0 (1 + w[:, 0])."""
    q, k, v = (_rand(i, (2, 3, 1, 8)) for i in range(3))
    w = _rand(3, (3, 8, 4))
    for kind in ("elu1",):
        o, _ = orc.prefill_quadratic(q, k, v, w, kind, 0.0)
        np.testing.assert_allclose(o, v * (1.0 + w[None, :, None, :, 0]), rtol=1e-13)


def test_equal_keys_give_running_mean():
    """All k_j equal: every weight for query i is the same, so la_i is the mean of v_0..v_i."""
    T, d = 33, 6
    q, v = _rand(0, (1, 2, T, d)), _rand(1, (1, 2, T, d))
    k = np.broadcast_to(_rand(2, (1, 2, 1, d)), (1, 2, T, d)).copy()
    w = np.zeros((2, d, 3))
    mean = np.cumsum(v, axis=2) / np.arange(1, T + 1)[None, None, :, None]
    for fn in (orc.prefill_quadratic, orc.prefill_recurrent):
        o, _ = fn(q, k, v, w, "elu1", 0.0)
        np.testing.assert_allclose(o, mean, rtol=1e-12, atol=1e-13)


def test_convex_combination_bounds_and_scale_invariance():
    T, d = 50, 8
    q, k, v = (_rand(i + 10, (2, 2, T, d)) for i in range(3))
    w = np.zeros((2, d, 3))
    o, _ = orc.prefill_quadratic(q, k, v, w, "elu1", 0.0)
    lo = np.minimum.accumulate(v, axis=2)
    hi = np.maximum.accumulate(v, axis=2)
    assert np.all(o >= lo - 1e-12) and np.all(o <= hi + 1e-12)
    # ReLU is positively homogeneous: scaling q leaves the ratio unchanged (eps = 0)
    q = np.abs(q) + 0.1
    k = np.abs(k) + 0.1
    o1, _ = orc.prefill_quadratic(q, k, v, w, "relu", 0.0)
    o2, _ = orc.prefill_quadratic(3.7 * q, k, v, w, "relu", 0.0)
    np.testing.assert_allclose(o1, o2, rtol=1e-12)


# ---------------------------------------------------------------- brute force
def _phi_scalar(x, kind):
    import math
    if kind == "relu":
        return max(x, 0.0)
    return x + 1.0 if x > 0 else math.exp(x)


def _brute(q, k, v, w, kind, eps):
    """Scalar loops over every index of the definition; nothing vectorised."""
    B, H, T, d = q.shape
    W = w.shape[2]
    o = np.zeros((B, H, T, d))
    for b in range(B):
        for h in range(H):
            for i in range(T):
                den = 0.0
                num = [0.0] * d
                for j in range(i + 1):
                    a = 0.0
                    for e in range(d):
                        a += _phi_scalar(q[b, h, i, e], kind) * _phi_scalar(k[b, h, j, e], kind)
                    den += a
                    for c in range(d):
                        num[c] += a * v[b, h, j, c]
                for c in range(d):
                    conv = 0.0
                    for t in range(W):
                        if i - t >= 0:
                            conv += w[h, c, t] * v[b, h, i - t, c]
                    o[b, h, i, c] = num[c] / (den + eps) + conv
    return o


@pytest.mark.parametrize("kind,eps", [("elu1", 0.0), ("relu", 1e-6)])
def test_brute_force_tiny(kind, eps):
    for T, d, W in ((1, 1, 1), (2, 1, 2), (4, 2, 3), (5, 3, 5), (7, 2, 9)):
        q, k, v = (_rand(100 + i + T, (2, 2, T, d)) for i in range(3))
        w = _rand(7, (2, d, W))
        want = _brute(q, k, v, w, kind, eps)
        for fn in (orc.prefill_quadratic, orc.prefill_recurrent):
            o, _ = fn(q, k, v, w, kind, eps)
            np.testing.assert_allclose(o, want, rtol=1e-11, atol=1e-12)


def test_exact_rational_example():
    """ReLU with small integer inputs: compare with exact Fraction arithmetic."""
    rs = np.random.default_rng(5)
    T, d = 6, 3
    q = rs.integers(0, 4, (1, 1, T, d)).astype(np.float64)
    k = rs.integers(1, 4, (1, 1, T, d)).astype(np.float64)
    v = rs.integers(-3, 4, (1, 1, T, d)).astype(np.float64)
    q[0, 0, :, 0] += 1
    w = np.zeros((1, d, 1))
    o, _ = orc.prefill_quadratic(q, k, v, w, "relu", 0.0)
    for i in range(T):
        den = Fraction(0)
        num = [Fraction(0)] * d
        for j in range(i + 1):
            a = sum(Fraction(int(q[0, 0, i, e])) * Fraction(int(k[0, 0, j, e])) for e in range(d))
            den += a
            num = [num[c] + a * int(v[0, 0, j, c]) for c in range(d)]
        for c in range(d):
            assert abs(o[0, 0, i, c] - float(num[c] / den)) < 1e-13


# ---------------------------------------------------------------- convolution against a library routine
@pytest.mark.parametrize("W", [1, 2, 3, 5, 32])
def test_conv_matches_library_causal_depthwise_conv1d(W):
    B, H, T, d = 2, 3, 40, 5
    v = _rand(1, (B, H, T, d))
    w = _rand(2, (H, d, W))
    got = orc.causal_dwconv(v, w, np.zeros((B, H, W - 1, d)))
    # library: channels = H*d, left padding W-1, cross-correlation => flip taps
    x = torch.from_numpy(v).permute(0, 1, 3, 2).reshape(B, H * d, T)
    x = torch.nn.functional.pad(x, (W - 1, 0))
    kern = torch.from_numpy(w).reshape(H * d, 1, W).flip(-1)
    want = torch.nn.functional.conv1d(x, kern, groups=H * d).reshape(B, H, d, T).permute(0, 1, 3, 2).numpy()
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)


def test_conv_special_cases():
    q, k, v = (_rand(i, (1, 2, 20, 4)) for i in range(3))
    o0, _ = orc.prefill_quadratic(q, k, v, np.zeros((2, 4, 3)), "elu1", 0.0)
    o1, _ = orc.prefill_quadratic(q, k, v, np.ones((2, 4, 1)), "elu1", 0.0)
    np.testing.assert_allclose(o1, o0 + v, rtol=1e-13)
    # a single delayed tap reproduces a shifted copy of v
    w = np.zeros((2, 4, 3))
    w[:, :, 2] = 1.0
    o2, _ = orc.prefill_quadratic(q, k, v, w, "elu1", 0.0)
    shifted = np.concatenate([np.zeros((1, 2, 2, 4)), v[:, :, :-2]], axis=2)
    np.testing.assert_allclose(o2, o0 + shifted, rtol=1e-13)


# ---------------------------------------------------------------- agreement of the three forms
@pytest.mark.parametrize("kind,eps", [("elu1", 0.0), ("relu", 1e-6)])
@pytest.mark.parametrize("T", [1, 63, 200])
def test_three_forms_agree(kind, eps, T):
    B, H, d, W = 2, 2, 16, 4
    q, k, v = (_rand(i + T, (B, H, T, d)) for i in range(3))
    w = _rand(9, (H, d, W))
    oq, sq = orc.prefill_quadratic(q, k, v, w, kind, eps)
    orr, sr = orc.prefill_recurrent(q, k, v, w, kind, eps)
    np.testing.assert_allclose(orr, oq, rtol=1e-11, atol=1e-12)
    for C in (1, 16, 64, 77, 256):
        oc, sc = orc.prefill_chunked(q, k, v, w, kind, eps, C)
        np.testing.assert_allclose(oc, oq, rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(sc.S, sq.S, rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(sc.z, sq.z, rtol=1e-12)
        np.testing.assert_array_equal(sc.win, sq.win)
    np.testing.assert_allclose(sr.S, sq.S, rtol=1e-11, atol=1e-12)
    np.testing.assert_array_equal(sr.win, sq.win)
    assert np.all(sq.pos == T) and np.all(sr.pos == T)


def test_continuation_equals_one_shot():
    B, H, T, d, W = 1, 2, 90, 8, 5
    q, k, v = (_rand(i + 40, (B, H, T, d)) for i in range(3))
    w = _rand(3, (H, d, W))
    o, st = orc.prefill_quadratic(q, k, v, w, "elu1", 0.0)
    for T1 in (1, 3, 50, 89):
        o1, s1 = orc.prefill_quadratic(q[:, :, :T1], k[:, :, :T1], v[:, :, :T1], w, "elu1", 0.0)
        o2, s2 = orc.prefill_chunked(q[:, :, T1:], k[:, :, T1:], v[:, :, T1:], w, "elu1", 0.0, 16, s1)
        o3, s3 = orc.prefill_quadratic(q[:, :, T1:], k[:, :, T1:], v[:, :, T1:], w, "elu1", 0.0, s1)
        np.testing.assert_allclose(np.concatenate([o1, o2], axis=2), o, rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(np.concatenate([o1, o3], axis=2), o, rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(s2.S, st.S, rtol=1e-11, atol=1e-12)
        np.testing.assert_array_equal(s2.win, st.win)
        assert s2.pos[0] == T


# ---------------------------------------------------------------- causality (no leakage from later tokens)
@pytest.mark.parametrize("W", [3, 32])
def test_no_future_leakage(W):
    B, H, T, d = 1, 2, 48, 8
    q, k, v = (_rand(i + 60, (B, H, T, d)) for i in range(3))
    w = _rand(4, (H, d, W))
    o, _ = orc.prefill_quadratic(q, k, v, w, "elu1", 0.0)
    j = 20
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    q2[:, :, j] += 1.0
    k2[:, :, j] -= 2.0
    v2[:, :, j] *= 3.0
    for fn in (orc.prefill_quadratic, orc.prefill_recurrent):
        o2, _ = fn(q2, k2, v2, w, "elu1", 0.0)
        o1, _ = fn(q, k, v, w, "elu1", 0.0)
        np.testing.assert_array_equal(o2[:, :, :j], o1[:, :, :j])
        assert np.all(o2[:, :, j] != o1[:, :, j])


# ---------------------------------------------------------------- trees
def _tree_case(seed, B=2, H=2, N=12, d=8, W=3, T0=10, kind="elu1", eps=0.0):
    q0, k0, v0 = (_rand(seed + i, (B, H, T0, d)) for i in range(3))
    w = _rand(seed + 5, (H, d, W))
    _, st = orc.prefill_quadratic(q0, k0, v0, w, kind, eps)
    q, k, v = (_rand(seed + 10 + i, (B, H, N, d)) for i in range(3))
    parent = np.stack([wl.random_tree(np.random.default_rng(seed + b), N, 5, 4) for b in range(B)])
    return st, q, k, v, parent, w


@pytest.mark.parametrize("kind,eps,W", [("elu1", 0.0, 3), ("relu", 1e-6, 5), ("elu1", 0.0, 1), ("elu1", 0.0, 9)])
def test_tree_equals_sequential_decode_on_every_path(kind, eps, W):
    st, q, k, v, parent, w = _tree_case(7, W=W, kind=kind, eps=eps)
    o = orc.verify_tree(q, k, v, parent, w, kind, eps, st)
    B, H, N, d = q.shape
    for b in range(B):
        for n in range(N):
            # walk the path in the test itself
            path, m = [], n
            while m >= 0:
                path.append(m)
                m = int(parent[b, m])
            path.reverse()
            s = orc.State(st.S[b:b + 1].copy(), st.z[b:b + 1].copy(), st.win[b:b + 1].copy(), st.pos[b:b + 1].copy())
            for m in path:
                last, s = orc.decode_step(q[b:b + 1, :, m], k[b:b + 1, :, m], v[b:b + 1, :, m], w, kind, eps, s)
            np.testing.assert_allclose(o[b, :, n], last[0], rtol=1e-11, atol=1e-12)


def test_chain_tree_equals_prefill_continuation():
    st, q, k, v, _, w = _tree_case(11, N=9, W=4)
    parent = np.stack([wl.chain_tree(9)] * q.shape[0])
    o = orc.verify_tree(q, k, v, parent, w, "elu1", 0.0, st)
    o2, _ = orc.prefill_quadratic(q, k, v, w, "elu1", 0.0, st)
    np.testing.assert_allclose(o, o2, rtol=1e-11, atol=1e-12)


def test_siblings_do_not_see_each_other():
    """Sec. 4.2: at time step t1 a candidate convolves over {t0, t1} of its own chain, never a sibling."""
    st, q, k, v, _, w = _tree_case(13, B=1, N=4, W=3)
    parent = np.array([[-1, 0, 0, 2]], dtype=np.int32)     # 1 and 2 are siblings; 3 hangs under 2
    o = orc.verify_tree(q, k, v, parent, w, "elu1", 0.0, st)
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    q2[:, :, 1] += 5.0
    k2[:, :, 1] -= 1.0
    v2[:, :, 1] *= -4.0
    o2 = orc.verify_tree(q2, k2, v2, parent, w, "elu1", 0.0, st)
    for n in (0, 2, 3):
        np.testing.assert_array_equal(o2[:, :, n], o[:, :, n])
    assert np.all(o2[:, :, 1] != o[:, :, 1])
    # removing the sibling altogether leaves the others unchanged as well
    keep = [0, 2, 3]
    parent3 = np.array([[-1, 0, 1]], dtype=np.int32)
    o3 = orc.verify_tree(q[:, :, keep], k[:, :, keep], v[:, :, keep], parent3, w, "elu1", 0.0, st)
    np.testing.assert_allclose(o3, o[:, :, keep], rtol=1e-13)


def test_relabelling_invariance():
    st, q, k, v, parent, w = _tree_case(17, B=1, N=10)
    o = orc.verify_tree(q, k, v, parent, w, "elu1", 0.0, st)
    # another topological order: sort nodes by (depth, -index)
    depth = wl.tree_depths(parent[0])
    order = sorted(range(10), key=lambda n: (depth[n], -n))
    new_of = {old: new for new, old in enumerate(order)}
    parent2 = np.array([[new_of[int(parent[0, old])] if parent[0, old] >= 0 else -1 for old in order]], dtype=np.int32)
    o2 = orc.verify_tree(q[:, :, order], k[:, :, order], v[:, :, order], parent2, w, "elu1", 0.0, st)
    np.testing.assert_allclose(o2, o[:, :, order], rtol=1e-12, atol=1e-13)


def test_verify_leaves_state_untouched_and_commit_equals_decode():
    st, q, k, v, parent, w = _tree_case(19, B=3, N=14, W=4)
    before = st.copy()
    orc.verify_tree(q, k, v, parent, w, "elu1", 0.0, st)
    for a, b in zip((st.S, st.z, st.win, st.pos), (before.S, before.z, before.win, before.pos)):
        np.testing.assert_array_equal(a, b)
    accept = np.array([13, -1, 5], dtype=np.int32)
    new, path, clen = orc.commit(k, v, parent, accept, "elu1", st, max_depth=6)
    for b in range(3):
        chain, m = [], int(accept[b])
        while m >= 0:
            chain.append(m)
            m = int(parent[b, m])
        chain.reverse()
        assert clen[b] == len(chain)
        assert list(path[b, :len(chain)]) == chain and np.all(path[b, len(chain):] == -1)
        s = orc.State(st.S[b:b + 1].copy(), st.z[b:b + 1].copy(), st.win[b:b + 1].copy(), st.pos[b:b + 1].copy())
        for m in chain:
            _, s = orc.decode_step(q[b:b + 1, :, m], k[b:b + 1, :, m], v[b:b + 1, :, m], w, "elu1", 0.0, s)
        np.testing.assert_allclose(new.S[b], s.S[0], rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(new.z[b], s.z[0], rtol=1e-13)
        np.testing.assert_array_equal(new.win[b], s.win[0])
        assert new.pos[b] == s.pos[0]
    # accept = -1 is a no-op
    np.testing.assert_array_equal(new.S[1], st.S[1])
    assert new.pos[1] == st.pos[1]


# ---------------------------------------------------------------------- greedy acceptance
def test_hand_example_accept():
    g = json.load(open(os.path.join(GOLD, "hand_example_accept.json")))
    parent = np.array([g["parent"]], dtype=np.int32)
    draft = np.array([g["draft_token"]], dtype=np.int32)
    pred = np.array([g["pred"]], dtype=np.int32)
    node, length, nxt = orc.accept_greedy(parent, draft, np.array([g["pred_root"]]), pred)
    assert (int(node[0]), int(length[0]), int(nxt[0])) == (g["accept_node"], g["accept_len"], g["next_token"])
    node, length, nxt = orc.accept_greedy(parent, draft, np.array([g["pred_root_none"]]), pred)
    assert (int(node[0]), int(length[0]), int(nxt[0])) == (g["accept_node_none"], g["accept_len_none"],
                                                           g["next_token_none"])


def _accepted_by_path_enumeration(parent, draft, pred_root, pred):
    """The definition read the other way round: for every node spell out its root-to-node path and check every
    token on it against the verifier's prediction at the position before it."""
    N = len(parent)
    best, best_len = -1, 0
    for n in range(N):
        path = orc.ancestors_or_self(parent, n)
        expected = [pred_root] + [pred[m] for m in path[:-1]]
        if all(int(draft[m]) == int(e) for m, e in zip(path, expected)) and len(path) > best_len:
            best, best_len = n, len(path)
    return best, best_len, (int(pred[best]) if best >= 0 else int(pred_root))


@pytest.mark.parametrize("vocab", [2, 3, 6])
def test_accept_brute_force_over_all_paths(vocab):
    for rnd in range(6):
        parent, _ = wl.tree_batch(11, rnd, 5, 24, max_depth=6, max_fanout=3)
        draft, pred_root, pred = wl.token_batch(11, rnd, 5, 24, vocab=vocab)
        node, length, nxt = orc.accept_greedy(parent, draft, pred_root, pred)
        for b in range(5):
            assert (int(node[b]), int(length[b]), int(nxt[b])) == _accepted_by_path_enumeration(
                parent[b], draft[b], int(pred_root[b]), pred[b])


def test_accept_on_a_chain_stops_at_the_first_mismatch():
    N = 12
    parent = wl.chain_tree(N)[None]
    pred_root = np.array([5])
    pred = np.arange(100, 100 + N, dtype=np.int32)[None]               # after node n the verifier says 100 + n
    draft = np.concatenate([[5], pred[0, :-1]]).astype(np.int32)[None]  # the drafter guessed everything right
    node, length, nxt = orc.accept_greedy(parent, draft, pred_root, pred)
    assert (int(node[0]), int(length[0]), int(nxt[0])) == (N - 1, N, 100 + N - 1)
    for miss in (0, 4, N - 1):                                          # one wrong draft at position `miss`
        d = draft.copy()
        d[0, miss] = -7
        node, length, nxt = orc.accept_greedy(parent, d, pred_root, pred)
        assert (int(node[0]), int(length[0])) == (miss - 1, miss)
        assert int(nxt[0]) == (5 if miss == 0 else 100 + miss - 1)


def test_accepted_chain_is_accepted_and_cannot_be_extended():
    parent, _ = wl.tree_batch(12, 0, 8, 40, max_depth=6, max_fanout=3)
    draft, pred_root, pred = wl.token_batch(12, 0, 8, 40, vocab=3)
    node, length, nxt = orc.accept_greedy(parent, draft, pred_root, pred)
    depths = [wl.tree_depths(parent[b]) for b in range(8)]
    for b in range(8):
        a = int(node[b])
        if a >= 0:
            path = orc.ancestors_or_self(parent[b], a)
            assert len(path) == int(length[b]) == depths[b][a]
            assert int(draft[b][path[0]]) == int(pred_root[b])
            for m, c in zip(path[:-1], path[1:]):
                assert int(draft[b][c]) == int(pred[b][m])
            # no child of the accepted node carries the token the verifier wants next
            assert not any(parent[b][c] == a and draft[b][c] == nxt[b] for c in range(40))
        else:
            assert not any(parent[b][c] == -1 and draft[b][c] == pred_root[b] for c in range(40))


def test_bad_trees_are_rejected():
    st, q, k, v, parent, w = _tree_case(23, B=1, N=5)
    bad = parent.copy()
    bad[0, 2] = 3
    with pytest.raises(ValueError):
        orc.verify_tree(q, k, v, bad, w, "elu1", 0.0, st)
    with pytest.raises(ValueError):
        orc.commit(k, v, parent, np.array([5]), "elu1", st, max_depth=8)


# ---------------------------------------------------------------- planted mistakes are caught
def test_pins_catch_planted_mistakes(monkeypatch):
    """Plant typical slips in the oracle and check that a pin notices each."""
    g = json.load(open(os.path.join(GOLD, "hand_example_relu.json")))
    q, k, v = (np.array(g[n], dtype=np.float64)[None, None] for n in "qkv")
    w = np.array(g["w"])[None]
    want = np.array(g["o"])

    def off(fn):
        o, _ = fn()
        return float(np.max(np.abs(o[0, 0] - want)))

    # (a) strict instead of inclusive causal mask
    real_tril = np.tril
    monkeypatch.setattr(orc.np, "tril", lambda a, k=0: real_tril(a, -1))
    with np.errstate(all="ignore"):
        assert not off(lambda: orc.prefill_quadratic(q, k, v, w, "relu", 0.0)) < 1e-6
    monkeypatch.undo()
    # (b) transposed state product in the recurrence
    real = orc.decode_step

    def swapped(q_, k_, v_, w_, kind, eps, st):
        return real(q_, v_, k_, w_, kind, eps, st)
    assert off(lambda: (np.stack([swapped(q[:, :, i], k[:, :, i], v[:, :, i], w, "relu", 0.0,
                                          orc.empty_state(1, 1, 2, 2))[0] for i in range(3)], axis=2), None)) > 1e-6
    # (c) reversed taps
    assert off(lambda: orc.prefill_quadratic(q, k, v, w[:, :, ::-1], "relu", 0.0)) > 1e-6
    # (d) acceptance: the verifier's predictions attached to the wrong nodes (shifted by one) change the hand-worked
    #     result, and the tie of that example (nodes 5 and 6, both at depth 3) goes to the smaller index
    g = json.load(open(os.path.join(GOLD, "hand_example_accept.json")))
    parent = np.array([g["parent"]], dtype=np.int32)
    draft = np.array([g["draft_token"]], dtype=np.int32)
    pred = np.array([g["pred"]], dtype=np.int32)
    node, length, _ = orc.accept_greedy(parent, draft, np.array([g["pred_root"]]), np.roll(pred, 1, axis=1))
    assert (int(node[0]), int(length[0])) != (g["accept_node"], g["accept_len"])
    node, _, _ = orc.accept_greedy(parent, draft, np.array([g["pred_root"]]), pred)
    assert int(node[0]) == 5
