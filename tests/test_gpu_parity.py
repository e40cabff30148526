"""Parity of the CUDA path (through the C boundary) with the float64 oracle, element by element."""
import numpy as np
import pytest
import torch

from oracle import la_oracle as orc
from paper_2406_07368_b200 import binding, workloads as wl
from tests._util import TOL, rel_err

pytestmark = pytest.mark.gpu


def dev(x, io):
    return torch.from_numpy(np.ascontiguousarray(x)).to(binding.TORCH_DTYPE[io]).cuda()


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64) if t.is_floating_point() else t.cpu().numpy()


def oracle_state_to_dev(st, io):
    return binding.State(torch.from_numpy(st.S).float().cuda(), torch.from_numpy(st.z).float().cuda(),
                         dev(st.win.astype(np.float32), io), torch.from_numpy(st.pos).cuda())


def check_state(got: binding.State, want: orc.State, tol, exact_window=True):
    assert rel_err(host(got.S), want.S) < tol
    assert rel_err(host(got.z), want.z) < tol
    if exact_window:
        np.testing.assert_array_equal(host(got.win), want.win)
    np.testing.assert_array_equal(host(got.pos), want.pos)


def make(io, B, H, d, T, W, seed, scale=1.0):
    q, k, v = wl.qkv(seed, (B, H, T, d), scale, io)
    w = wl.conv_weights(seed, H, d, W)
    return q, k, v, w


# ------------------------------------------------------------------ prefill
@pytest.mark.parametrize("kernel", [0, 1])
@pytest.mark.parametrize("io,d,phi,eps,W,T", [
    ("f32", 64, "elu1", 0.0, 3, 256),
    ("f32", 128, "relu", 1e-6, 5, 70),
    ("bf16", 128, "elu1", 0.0, 3, 1),
    ("bf16", 128, "elu1", 0.0, 3, 127),
    ("bf16", 128, "elu1", 0.0, 3, 128),
    ("bf16", 128, "elu1", 0.0, 3, 129),
    ("bf16", 128, "elu1", 0.0, 3, 700),
    ("bf16", 128, "relu", 1e-6, 5, 333),
    ("bf16", 64, "elu1", 0.0, 3, 200),
    ("bf16", 128, "elu1", 0.0, 32, 150),
    ("bf16", 128, "elu1", 0.0, 26, 300),
    ("bf16", 128, "relu", 1e-6, 27, 300),
    ("bf16", 128, "elu1", 0.0, 1, 150),
])
def test_prefill_matches_oracle(kernel, io, d, phi, eps, W, T):
    B, H = 2, 3
    scale = 1.0 if io == "f32" else d ** -0.5
    q, k, v, w = make(io, B, H, d, T, W, seed=T + W, scale=scale)
    ctx = binding.Context(H, d, W, phi, eps, io)
    ctx.la_set_prefill_kernel(kernel)
    st = ctx.new_state(B)
    st.S.fill_(7.0)          # a fresh prefill must ignore whatever the buffers hold
    st.pos.fill_(99)
    o = ctx.la_prefill(dev(q, io), dev(k, io), dev(v, io), dev(w, "f32"), st, init_state=False)
    want, wst = orc.prefill_quadratic(q, k, v, w, phi, eps)
    assert ctx.la_last_device_status() == binding.LA_OK
    assert rel_err(host(o), want) < TOL[io]
    check_state(st, wst, TOL[io])


@pytest.mark.parametrize("kernel", [0, 1])
@pytest.mark.parametrize("io,T1,T2", [("f32", 50, 77), ("bf16", 1, 200), ("bf16", 130, 129), ("bf16", 255, 2)])
def test_prefill_continuation(kernel, io, T1, T2):
    B, H, d, W = 1, 2, 128, 4
    q, k, v, w = make(io, B, H, d, T1 + T2, W, seed=5, scale=0.5)
    ctx = binding.Context(H, d, W, "elu1", 0.0, io)
    ctx.la_set_prefill_kernel(kernel)
    st = ctx.new_state(B)
    cut = lambda x, a, b: dev(x[:, :, a:b], io)
    o1 = ctx.la_prefill(cut(q, 0, T1), cut(k, 0, T1), cut(v, 0, T1), dev(w, "f32"), st, init_state=False)
    o2 = ctx.la_prefill(cut(q, T1, T1 + T2), cut(k, T1, T1 + T2), cut(v, T1, T1 + T2), dev(w, "f32"), st,
                        init_state=True)
    want, wst = orc.prefill_quadratic(q, k, v, w, "elu1", 0.0)
    assert rel_err(np.concatenate([host(o1), host(o2)], axis=2), want) < TOL[io]
    check_state(st, wst, TOL[io])


def test_prefill_more_chains_than_sms():
    """160 chains on 148 SMs: the chains of the second wave start when CTAs of the first one have left."""
    io, B, H, d, W, T = "bf16", 5, 32, 128, 3, 300
    q, k, v, w = make(io, B, H, d, T, W, seed=77, scale=d ** -0.5)
    ctx = binding.Context(H, d, W, "elu1", 0.0, io)
    st = ctx.new_state(B)
    o = ctx.la_prefill(dev(q, io), dev(k, io), dev(v, io), dev(w, "f32"), st)
    assert ctx.la_last_device_status() == binding.LA_OK
    for b, h in ((0, 0), (2, 17), (4, 19), (4, 31)):                     # (4, 19) and (4, 31): chains 147 and 159
        sl = (slice(b, b + 1), slice(h, h + 1))
        want, wst = orc.prefill_quadratic(q[sl], k[sl], v[sl], w[h:h + 1], "elu1", 0.0)
        assert rel_err(host(o[sl]), want) < TOL[io], (b, h)
        assert rel_err(host(st.S[sl]), wst.S) < TOL[io] and rel_err(host(st.z[sl]), wst.z) < TOL[io]
        np.testing.assert_array_equal(host(st.win[sl]), wst.win)
    assert st.pos.tolist() == [T] * B


@pytest.mark.parametrize("W", [32, 9, 6])
@pytest.mark.parametrize("T1,T2,T3", [(20, 300, 9), (140, 17, 130), (3, 1, 260)])
def test_prefill_continuation_with_long_tap_windows(T1, T2, T3, W):
    """Windows that take the long epilogue (taps in groups of 8, one halo updated in place): the window carried
    between calls is longer than some of the pieces, 32 taps reach back across a whole 32-row block, and 9 and 6
    taps leave most of a group of 8 as zero padding."""
    io, B, H, d = "bf16", 2, 2, 128
    T = T1 + T2 + T3
    q, k, v, w = make(io, B, H, d, T, W, seed=15, scale=0.5)
    ctx = binding.Context(H, d, W, "elu1", 0.0, io)
    st = ctx.new_state(B)
    cut = lambda x, a, b: dev(x[:, :, a:b], io)
    outs, a = [], 0
    for i, n in enumerate((T1, T2, T3)):
        outs.append(ctx.la_prefill(cut(q, a, a + n), cut(k, a, a + n), cut(v, a, a + n), dev(w, "f32"), st,
                                   init_state=i > 0))
        a += n
    want, wst = orc.prefill_quadratic(q, k, v, w, "elu1", 0.0)
    assert ctx.la_last_device_status() == binding.LA_OK
    assert rel_err(np.concatenate([host(o) for o in outs], axis=2), want) < TOL[io]
    check_state(st, wst, TOL[io])


@pytest.mark.parametrize("T,W,phi,eps,init", [(2500, 3, "elu1", 0.0, False), (4099, 5, "relu", 1e-6, False),
                                              (3000, 4, "elu1", 0.0, True), (2048, 1, "elu1", 0.0, False),
                                              (2300, 32, "elu1", 0.0, True), (2200, 27, "relu", 1e-6, False)])
def test_prefill_sequence_split_with_workspace(T, W, phi, eps, init):
    """Few chains and a long sequence: with a workspace the sequence is cut into segments run as separate CTAs."""
    io, B, H, d = "bf16", 1, 2, 128
    q, k, v, w = make(io, B, H, d, T, W, seed=T, scale=d ** -0.5)
    ctx = binding.Context(H, d, W, phi, eps, io)
    need = ctx.la_prefill_workspace_bytes(B, T)
    assert need > 0
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    ctx.la_set_workspace(ws)
    st = ctx.new_state(B)
    ost = None
    if init:
        q0, k0, v0, _ = make(io, B, H, d, 70, W, seed=1, scale=d ** -0.5)
        _, ost = orc.prefill_quadratic(q0, k0, v0, w, phi, eps)
        st = oracle_state_to_dev(ost, io)
    n0 = ctx.la_launch_count()
    o = ctx.la_prefill(dev(q, io), dev(k, io), dev(v, io), dev(w, "f32"), st, init_state=init)
    assert ctx.la_launch_count() - n0 == 3                     # segment states, prefix, segments
    assert ctx.la_last_device_status() == binding.LA_OK
    want, wst = orc.prefill_chunked(q, k, v, w, phi, eps, 256, ost)
    assert rel_err(host(o), want) < TOL[io]
    check_state(st, wst, TOL[io])
    # without the workspace the same call runs one CTA per chain and agrees up to rounding order
    ctx.la_set_workspace(None)
    st2 = ctx.new_state(B) if not init else oracle_state_to_dev(ost, io)
    o2 = ctx.la_prefill(dev(q, io), dev(k, io), dev(v, io), dev(w, "f32"), st2, init_state=init)
    assert rel_err(host(o2), want) < TOL[io]
    assert rel_err(host(o2), host(o)) < TOL[io]
    assert torch.equal(st.win, st2.win) and torch.equal(st.pos, st2.pos)


def test_prefill_is_causal_bitwise():
    """Perturbing token j leaves every earlier output bit-identical (no leakage through the conv)."""
    io, B, H, d, T, W = "bf16", 1, 2, 128, 300, 8
    q, k, v, w = make(io, B, H, d, T, W, seed=11, scale=0.3)
    ctx = binding.Context(H, d, W, "elu1", 0.0, io)
    for kernel in (0, 1):
        ctx.la_set_prefill_kernel(kernel)
        o1 = ctx.la_prefill(dev(q, io), dev(k, io), dev(v, io), dev(w, "f32"), ctx.new_state(B))
        j = 200
        q2, k2, v2 = q.copy(), k.copy(), v.copy()
        q2[:, :, j] = wl.round_to_bf16(q2[:, :, j] + 1)
        k2[:, :, j] = wl.round_to_bf16(k2[:, :, j] - 1)
        v2[:, :, j] = wl.round_to_bf16(v2[:, :, j] * 3)
        o2 = ctx.la_prefill(dev(q2, io), dev(k2, io), dev(v2, io), dev(w, "f32"), ctx.new_state(B))
        assert torch.equal(o1[:, :, :j], o2[:, :, :j])
        assert not torch.equal(o1[:, :, j], o2[:, :, j])


# ------------------------------------------------------------------ decode
@pytest.mark.parametrize("io,d,phi,eps,W", [("f32", 64, "elu1", 0.0, 3), ("bf16", 128, "elu1", 0.0, 3),
                                            ("bf16", 128, "relu", 1e-6, 5), ("bf16", 64, "elu1", 0.0, 1),
                                            ("f32", 128, "elu1", 0.0, 32), ("bf16", 128, "elu1", 0.0, 2),
                                            ("bf16", 128, "elu1", 0.0, 4), ("bf16", 128, "relu", 1e-6, 8),
                                            ("bf16", 128, "elu1", 0.0, 9), ("bf16", 128, "elu1", 0.0, 17),
                                            ("bf16", 128, "elu1", 0.0, 32)])
def test_decode_matches_oracle(io, d, phi, eps, W):
    B, H, T0, steps = 3, 2, 40, 12
    q, k, v, w = make(io, B, H, d, T0, W, seed=21 + W, scale=0.7)
    ctx = binding.Context(H, d, W, phi, eps, io)
    _, ost = orc.prefill_quadratic(q, k, v, w, phi, eps)
    st = oracle_state_to_dev(ost, io)
    for s in range(steps):
        qs, ks, vs = wl.qkv(100 + s, (B, H, d), 0.7, io)
        o = ctx.la_decode_step(dev(qs, io), dev(ks, io), dev(vs, io), dev(w, "f32"), st)
        want, ost = orc.decode_step(qs, ks, vs, w, phi, eps, ost)
        assert rel_err(host(o), want) < TOL[io], s
    check_state(st, ost, TOL[io])


def test_prefill_then_decode_equals_longer_prefill():
    io, B, H, d, W, T, extra = "bf16", 1, 2, 128, 3, 140, 5
    q, k, v, w = make(io, B, H, d, T + extra, W, seed=31, scale=0.5)
    ctx = binding.Context(H, d, W, "elu1", 0.0, io)
    st = ctx.new_state(B)
    ctx.la_prefill(dev(q[:, :, :T], io), dev(k[:, :, :T], io), dev(v[:, :, :T], io), dev(w, "f32"), st)
    outs = [ctx.la_decode_step(dev(q[:, :, T + i], io), dev(k[:, :, T + i], io), dev(v[:, :, T + i], io),
                               dev(w, "f32"), st) for i in range(extra)]
    want, wst = orc.prefill_quadratic(q, k, v, w, "elu1", 0.0)
    got = np.stack([host(o) for o in outs], axis=2)
    assert rel_err(got, want[:, :, T:]) < TOL[io]
    check_state(st, wst, TOL[io])


# ------------------------------------------------------------------ verify + commit
def tree_case(io, B, H, d, N, W, seed, phi="elu1", eps=0.0, chain=False):
    q0, k0, v0, w = make(io, B, H, d, 30, W, seed=seed, scale=0.7)
    _, ost = orc.prefill_quadratic(q0, k0, v0, w, phi, eps)
    q, k, v = wl.qkv(seed + 1, (B, H, N, d), 0.7, io)
    if chain:
        parent = np.stack([wl.chain_tree(N)] * B)
    else:
        parent = np.stack([wl.random_tree(wl.rng(seed, 4, 0, b), N, 5, 4) for b in range(B)]).astype(np.int32)
    return ost, q, k, v, parent, w


@pytest.mark.parametrize("io,d,N,W,phi,eps,chain", [
    ("bf16", 128, 64, 3, "elu1", 0.0, False), ("bf16", 128, 37, 5, "relu", 1e-6, False),
    ("f32", 64, 4, 3, "elu1", 0.0, True), ("bf16", 64, 64, 3, "elu1", 0.0, False),
    ("bf16", 128, 1, 3, "elu1", 0.0, False), ("f32", 128, 64, 9, "elu1", 0.0, False),
    ("bf16", 128, 20, 32, "elu1", 0.0, True), ("bf16", 128, 16, 1, "elu1", 0.0, False),
    ("bf16", 128, 64, 4, "relu", 1e-6, True), ("bf16", 128, 37, 2, "relu", 1e-6, False),
    ("bf16", 128, 50, 4, "elu1", 0.0, False), ("bf16", 128, 33, 4, "elu1", 1e-6, True),
    ("bf16", 128, 64, 8, "elu1", 0.0, False), ("bf16", 128, 64, 32, "elu1", 1e-6, False),
    ("bf16", 128, 3, 6, "relu", 1e-6, True), ("bf16", 128, 64, 17, "relu", 0.0, True)])
@pytest.mark.parametrize("kernel", [0, 1])
def test_verify_matches_oracle_and_leaves_state_untouched(kernel, io, d, N, W, phi, eps, chain):
    B, H = 3, 2
    ost, q, k, v, parent, w = tree_case(io, B, H, d, N, W, seed=41 + N, phi=phi, eps=eps, chain=chain)
    ctx = binding.Context(H, d, W, phi, eps, io, max_nodes=64, max_depth=64)
    ctx.la_set_prefill_kernel(kernel)
    st = oracle_state_to_dev(ost, io)
    before = st.clone()
    o = ctx.la_verify_tree(dev(q, io), dev(k, io), dev(v, io), torch.from_numpy(parent).cuda(), dev(w, "f32"), st)
    assert ctx.la_last_device_status() == binding.LA_OK
    want = orc.verify_tree(q, k, v, parent, w, phi, eps, ost)
    assert rel_err(host(o), want) < TOL[io]
    for a, b in ((st.S, before.S), (st.z, before.z), (st.win, before.win), (st.pos, before.pos)):
        assert torch.equal(a, b)


def test_verify_every_tree_size():
    """N = 1 .. 64 on the tensor-core path (rows past N are padding inside the kernel)."""
    io, B, H, d, W = "bf16", 1, 2, 128, 3
    ctx = binding.Context(H, d, W, "elu1", 0.0, io, max_nodes=64, max_depth=64)
    ost, q, k, v, _, w = tree_case(io, B, H, d, 64, W, seed=123)
    st = oracle_state_to_dev(ost, io)
    for N in range(1, 65):
        parent = np.stack([wl.random_tree(wl.rng(123, 4, N, 0), N, 6, 3)]).astype(np.int32)
        qn, kn, vn = (np.ascontiguousarray(x[:, :, :N]) for x in (q, k, v))
        o = ctx.la_verify_tree(dev(qn, io), dev(kn, io), dev(vn, io), torch.from_numpy(parent).cuda(), dev(w, "f32"), st)
        want = orc.verify_tree(qn, kn, vn, parent, w, "elu1", 0.0, ost)
        assert rel_err(host(o), want) < TOL[io], N
    assert ctx.la_last_device_status() == binding.LA_OK


def test_prefill_lengths_around_the_tile_edges():
    io, B, H, d, W = "bf16", 1, 2, 128, 3
    ctx = binding.Context(H, d, W, "elu1", 0.0, io)
    q, k, v, w = make(io, B, H, d, 400, W, seed=321, scale=d ** -0.5)
    for T in (1, 2, 3, 63, 64, 65, 126, 127, 128, 129, 130, 255, 256, 257, 383, 384, 385):
        st = ctx.new_state(B)
        cut = lambda x: dev(x[:, :, :T], io)
        o = ctx.la_prefill(cut(q), cut(k), cut(v), dev(w, "f32"), st)
        want, wst = orc.prefill_quadratic(q[:, :, :T], k[:, :, :T], v[:, :, :T], w, "elu1", 0.0)
        assert rel_err(host(o), want) < TOL[io], T
        check_state(st, wst, TOL[io])
    assert ctx.la_last_device_status() == binding.LA_OK


@pytest.mark.parametrize("W", [4, 7])
def test_verify_more_units_than_sms_with_one_bad_tree(W):
    """Several units per persistent CTA; one sequence in the middle carries an invalid tree."""
    io, B, H, d, N = "bf16", 48, 8, 128, 64
    ost, q, k, v, parent, w = tree_case(io, B, H, d, N, W, seed=97, phi="relu", eps=1e-6)
    ctx = binding.Context(H, d, W, "relu", 1e-6, io, max_nodes=64, max_depth=64)
    st = oracle_state_to_dev(ost, io)
    want = orc.verify_tree(q, k, v, parent, w, "relu", 1e-6, ost)
    o = ctx.la_verify_tree(dev(q, io), dev(k, io), dev(v, io), torch.from_numpy(parent).cuda(), dev(w, "f32"), st)
    assert ctx.la_last_device_status() == binding.LA_OK
    assert rel_err(host(o), want) < TOL[io]
    for b in (0, 20, 47):                                  # per sequence, so that one wrong unit cannot hide
        assert rel_err(host(o[b]), want[b]) < TOL[io]
    bad = parent.copy()
    bad[20, 9] = 9                                         # a node that is its own parent
    out = torch.full((B, H, N, d), 123.0, dtype=torch.bfloat16, device="cuda")
    ctx.la_verify_tree(dev(q, io), dev(k, io), dev(v, io), torch.from_numpy(bad).cuda(), dev(w, "f32"), st, out=out)
    assert ctx.la_last_device_status() == binding.LA_ERR_BAD_TREE
    assert torch.all(out[20] == 123.0)
    good = [b for b in range(B) if b != 20]
    assert rel_err(host(out[good]), want[good]) < TOL[io]


@pytest.mark.parametrize("B,H,W", [(50, 4, 3), (149, 1, 3), (37, 8, 4), (51, 4, 8), (64, 8, 3)])
def test_verify_unit_counts_around_the_number_of_sms(B, H, W):
    """Unit counts just above, far above and at multiples of the number of SMs (148: 200 units, 149, 296, 204, 512):
    the persistent grid's last round is partly filled.  Every sequence is compared on its own and by channel half,
    and a bad tree in one of the last sequences leaves its outputs untouched."""
    io, d, N = "bf16", 128, 24
    ost, q, k, v, parent, w = tree_case(io, B, H, d, N, W, seed=300 + B, phi="elu1", eps=0.0)
    ctx = binding.Context(H, d, W, "elu1", 0.0, io, max_nodes=64, max_depth=64)
    st = oracle_state_to_dev(ost, io)
    before = st.clone()
    want = orc.verify_tree(q, k, v, parent, w, "elu1", 0.0, ost)
    o = ctx.la_verify_tree(dev(q, io), dev(k, io), dev(v, io), torch.from_numpy(parent).cuda(), dev(w, "f32"), st)
    assert ctx.la_last_device_status() == binding.LA_OK
    got = host(o)
    for b in range(B):
        assert rel_err(got[b], want[b]) < TOL[io], b
        for half in (slice(0, 64), slice(64, 128)):
            assert rel_err(got[b][..., half], want[b][..., half]) < TOL[io], (b, half)
    assert torch.equal(st.S, before.S) and torch.equal(st.win, before.win)
    bad = parent.copy()
    bad[B - 2, 5] = 7                                       # a parent after its child, in one of the last sequences
    out = torch.full((B, H, N, d), 123.0, dtype=torch.bfloat16, device="cuda")
    ctx.la_verify_tree(dev(q, io), dev(k, io), dev(v, io), torch.from_numpy(bad).cuda(), dev(w, "f32"), st, out=out)
    assert ctx.la_last_device_status() == binding.LA_ERR_BAD_TREE
    assert torch.all(out[B - 2] == 123.0)
    good = [b for b in range(B) if b != B - 2]
    assert rel_err(host(out[good]), want[good]) < TOL[io]


def test_verify_siblings_are_independent_bitwise():
    io, B, H, d, W = "bf16", 1, 2, 128, 3
    ost, q, k, v, _, w = tree_case(io, B, H, d, 4, W, seed=51)
    parent = np.array([[-1, 0, 0, 2]], dtype=np.int32)
    ctx = binding.Context(H, d, W, "elu1", 0.0, io)
    st = oracle_state_to_dev(ost, io)
    o1 = ctx.la_verify_tree(dev(q, io), dev(k, io), dev(v, io), torch.from_numpy(parent).cuda(), dev(w, "f32"), st)
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    q2[:, :, 1] = wl.round_to_bf16(q2[:, :, 1] + 2)
    k2[:, :, 1] = wl.round_to_bf16(k2[:, :, 1] - 1)
    v2[:, :, 1] = wl.round_to_bf16(v2[:, :, 1] * -4)
    o2 = ctx.la_verify_tree(dev(q2, io), dev(k2, io), dev(v2, io), torch.from_numpy(parent).cuda(), dev(w, "f32"), st)
    for n in (0, 2, 3):
        assert torch.equal(o1[:, :, n], o2[:, :, n])
    assert not torch.equal(o1[:, :, 1], o2[:, :, 1])


@pytest.mark.parametrize("io,d,N,W", [("bf16", 128, 64, 3), ("f32", 64, 10, 5), ("bf16", 128, 64, 8)])
def test_commit_matches_oracle_and_paths_are_exact(io, d, N, W):
    B, H = 4, 2
    ost, q, k, v, parent, w = tree_case(io, B, H, d, N, W, seed=61 + N)
    accept = np.array([wl.random_accept(wl.rng(7, 6, 0, b), parent[b]) for b in range(B)], dtype=np.int32)
    accept[1] = -1                                     # nothing accepted: a no-op
    ctx = binding.Context(H, d, W, "elu1", 0.0, io, max_nodes=64, max_depth=6)
    st = oracle_state_to_dev(ost, io)
    path, clen = ctx.la_commit(dev(k, io), dev(v, io), torch.from_numpy(parent).cuda(),
                               torch.from_numpy(accept).cuda(), st)
    assert ctx.la_last_device_status() == binding.LA_OK
    wst, wpath, wlen = orc.commit(k, v, parent, accept, "elu1", ost, max_depth=6)
    np.testing.assert_array_equal(host(path), wpath)
    np.testing.assert_array_equal(host(clen), wlen)
    check_state(st, wst, TOL[io])
    # and it equals decoding the path token by token on the GPU
    st2 = oracle_state_to_dev(ost, io)
    ctx1 = binding.Context(H, d, W, "elu1", 0.0, io)
    for b in range(B):
        sb = binding.State(st2.S[b:b + 1].clone(), st2.z[b:b + 1].clone(), st2.win[b:b + 1].clone(),
                           st2.pos[b:b + 1].clone())
        for n in wpath[b][:wlen[b]]:
            ctx1.la_decode_step(dev(q[b:b + 1, :, n], io), dev(k[b:b + 1, :, n], io), dev(v[b:b + 1, :, n], io),
                                dev(w, "f32"), sb)
        assert rel_err(host(sb.S), host(st.S[b:b + 1])) < 1e-5
        assert torch.equal(sb.win, st.win[b:b + 1]) and torch.equal(sb.pos, st.pos[b:b + 1])


@pytest.mark.parametrize("B,N,vocab,depth", [(7, 64, 3, 5), (1, 1, 2, 1), (13, 37, 2, 8), (4, 64, 1, 64)])
def test_accept_greedy_is_bit_exact(B, N, vocab, depth):
    ctx = binding.Context(2, 128, 3, "elu1", 0.0, "bf16", max_nodes=64, max_depth=64)
    for rnd in range(3):
        if depth == 64:
            parent = np.stack([wl.chain_tree(N)] * B)
        else:
            parent, _ = wl.tree_batch(21 + N, rnd, B, N, max_depth=depth, max_fanout=4)
        draft, pred_root, pred = wl.token_batch(21 + N, rnd, B, N, vocab=vocab)
        want = orc.accept_greedy(parent, draft, pred_root, pred)
        got = ctx.la_accept_greedy(*(torch.from_numpy(x).cuda() for x in (parent, draft, pred_root, pred)))
        assert ctx.la_last_device_status() == binding.LA_OK
        for g, w_ in zip(got, want):
            np.testing.assert_array_equal(g.cpu().numpy(), w_)


def test_accept_then_commit_matches_the_oracle():
    io, B, H, d, N, W = "bf16", 5, 2, 128, 32, 3
    ost, q, k, v, parent, w = tree_case(io, B, H, d, N, W, seed=91)
    draft, pred_root, pred = wl.token_batch(91, 0, B, N, vocab=2)
    ctx = binding.Context(H, d, W, "elu1", 0.0, io, max_nodes=64, max_depth=8)
    st = oracle_state_to_dev(ost, io)
    par = torch.from_numpy(parent).cuda()
    node, length, _ = ctx.la_accept_greedy(par, *(torch.from_numpy(x).cuda() for x in (draft, pred_root, pred)))
    path, clen = ctx.la_commit(dev(k, io), dev(v, io), par, node, st)
    assert ctx.la_last_device_status() == binding.LA_OK
    wnode, wlen, _ = orc.accept_greedy(parent, draft, pred_root, pred)
    wst, wpath, wclen = orc.commit(k, v, parent, wnode, "elu1", ost, max_depth=8)
    np.testing.assert_array_equal(host(clen), wlen)
    np.testing.assert_array_equal(host(path), wpath)
    assert torch.equal(clen, length)
    check_state(st, wst, TOL[io])


def test_accept_greedy_flags_bad_trees():
    B, N = 3, 8
    parent, _ = wl.tree_batch(5, 0, B, N)
    draft, pred_root, pred = wl.token_batch(5, 0, B, N, vocab=1)           # everything matches
    bad = parent.copy()
    bad[1, 2] = 6                                                          # parent after child
    ctx = binding.Context(2, 128, 3, "elu1", 0.0, "bf16", max_nodes=8)
    node, length, nxt = ctx.la_accept_greedy(*(torch.from_numpy(x).cuda() for x in (bad, draft, pred_root, pred)))
    assert ctx.la_last_device_status() == binding.LA_ERR_BAD_TREE
    assert int(node[1]) == -1 and int(length[1]) == 0 and int(nxt[1]) == int(pred_root[1])
    want = orc.accept_greedy(parent[[0, 2]], draft[[0, 2]], pred_root[[0, 2]], pred[[0, 2]])
    np.testing.assert_array_equal(node[[0, 2]].cpu().numpy(), want[0])
    ctx.la_clear_device_status()
    with pytest.raises(binding.LaError):
        ctx.la_accept_greedy(*(torch.zeros(1, 9, dtype=torch.int32, device="cuda") for _ in range(2)),
                             torch.zeros(1, dtype=torch.int32, device="cuda"),
                             torch.zeros(1, 9, dtype=torch.int32, device="cuda"))      # N > max_nodes


def test_bad_trees_set_the_status_word_and_write_nothing():
    io, B, H, d, N, W = "bf16", 2, 2, 128, 8, 3
    ost, q, k, v, parent, w = tree_case(io, B, H, d, N, W, seed=71)
    ctx = binding.Context(H, d, W, "elu1", 0.0, io, max_nodes=16, max_depth=2)
    st = oracle_state_to_dev(ost, io)
    bad = parent.copy()
    bad[1, 3] = 5                                      # parent after child in sequence 1
    out = torch.full((B, H, N, d), 123.0, dtype=torch.bfloat16, device="cuda")
    ctx.la_verify_tree(dev(q, io), dev(k, io), dev(v, io), torch.from_numpy(bad).cuda(), dev(w, "f32"), st, out=out)
    assert ctx.la_last_device_status() == binding.LA_ERR_BAD_TREE
    assert torch.all(out[1] == 123.0) and not torch.any(out[0] == 123.0)
    ctx.la_clear_device_status()
    assert ctx.la_last_device_status() == binding.LA_OK
    # accepted node outside the tree, and a path longer than max_depth
    chain = np.stack([wl.chain_tree(N)] * B)
    before = st.clone()
    for accept in ([N, 0], [0, 5]):
        path, clen = ctx.la_commit(dev(k, io), dev(v, io), torch.from_numpy(chain).cuda(),
                                   torch.tensor(accept, dtype=torch.int32).cuda(), st)
        assert ctx.la_last_device_status() == binding.LA_ERR_BAD_TREE
        ctx.la_clear_device_status()
        bad_b = 0 if accept[0] == N else 1
        assert torch.equal(st.S[bad_b], before.S[bad_b]) and torch.equal(st.pos[bad_b:bad_b + 1], before.pos[bad_b:bad_b + 1])
        st = before.clone()


def test_calls_recorded_in_a_cuda_graph_replay_bit_exactly():
    """Decode steps, a verification and a commit recorded once on a capturing stream, then replayed: the benchmark
    launches its steps this way.  Same kernels, same inputs: the results equal the eager ones bit for bit."""
    io, B, H, d, N, W = "bf16", 3, 4, 128, 16, 3
    ost, q, k, v, parent, w = tree_case(io, B, H, d, N, W, seed=83)
    accept = np.array([wl.random_accept(wl.rng(9, 6, 0, b), parent[b]) for b in range(B)], dtype=np.int32)
    ctx = binding.Context(H, d, W, "elu1", 0.0, io, max_nodes=16, max_depth=6)
    dq, dk, dv = dev(q, io), dev(k, io), dev(v, io)
    par, acc, dw = torch.from_numpy(parent).cuda(), torch.from_numpy(accept).cuda(), dev(w, "f32")

    def run(st, outs):
        for i in range(3):
            ctx.la_decode_step(dq[:, :, i].contiguous(), dk[:, :, i].contiguous(), dv[:, :, i].contiguous(), dw, st,
                               out=outs["dec"][i])
        ctx.la_verify_tree(dq, dk, dv, par, dw, st, out=outs["ver"])
        ctx.la_commit(dk, dv, par, acc, st, path_out=outs["path"], commit_len=outs["len"])

    def buffers():
        return {"dec": [torch.empty(B, H, d, dtype=torch.bfloat16, device="cuda") for _ in range(3)],
                "ver": torch.empty(B, H, N, d, dtype=torch.bfloat16, device="cuda"),
                "path": torch.empty(B, 6, dtype=torch.int32, device="cuda"),
                "len": torch.empty(B, dtype=torch.int32, device="cuda")}

    st_e, out_e = oracle_state_to_dev(ost, io), buffers()
    run(st_e, out_e)
    torch.cuda.synchronize()
    st_g, out_g = oracle_state_to_dev(ost, io), buffers()
    slices = [(dq[:, :, i].contiguous(), dk[:, :, i].contiguous(), dv[:, :, i].contiguous()) for i in range(3)]
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(3):
            ctx.la_decode_step(slices[i][0], slices[i][1], slices[i][2], dw, st_g, out=out_g["dec"][i])
        ctx.la_verify_tree(dq, dk, dv, par, dw, st_g, out=out_g["ver"])
        ctx.la_commit(dk, dv, par, acc, st_g, path_out=out_g["path"], commit_len=out_g["len"])
    fresh = oracle_state_to_dev(ost, io)                    # capture does not run anything: start from the same state
    for a, b in ((st_g.S, fresh.S), (st_g.z, fresh.z), (st_g.win, fresh.win), (st_g.pos, fresh.pos)):
        a.copy_(b)
    g.replay()
    torch.cuda.synchronize()
    assert ctx.la_last_device_status() == binding.LA_OK
    for i in range(3):
        assert torch.equal(out_e["dec"][i], out_g["dec"][i])
    assert torch.equal(out_e["ver"], out_g["ver"]) and torch.equal(out_e["path"], out_g["path"])
    assert torch.equal(out_e["len"], out_g["len"])
    for a, b in ((st_e.S, st_g.S), (st_e.z, st_g.z), (st_e.win, st_g.win), (st_e.pos, st_g.pos)):
        assert torch.equal(a, b)


def test_host_side_rejections():
    ctx = binding.Context(2, 128, 3, "elu1", 0.0, "bf16", max_nodes=8)
    st = ctx.new_state(1)
    x = torch.zeros(1, 2, 9, 128, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(2, 128, 3, device="cuda")
    par = torch.full((1, 9), -1, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.LaError) as e:
        ctx.la_verify_tree(x, x, x, par, w, st)        # N > max_nodes
    assert e.value.code == binding.LA_ERR_INVALID_ARG
    L = binding.lib()
    cs = st.c()
    import ctypes
    rc = L.la_prefill(ctx._h, 1, 9, x.data_ptr() + 2, x.data_ptr(), x.data_ptr(), w.data_ptr(), 0, ctypes.byref(cs),
                      x.data_ptr(), None)              # misaligned q
    assert rc == binding.LA_ERR_INVALID_ARG
    rc = L.la_prefill(ctx._h, 1, 0, x.data_ptr(), x.data_ptr(), x.data_ptr(), w.data_ptr(), 0, ctypes.byref(cs),
                      x.data_ptr(), None)              # T = 0
    assert rc == binding.LA_ERR_INVALID_ARG
    assert ctx.la_launch_count() == 0


# ------------------------------------------------------------------ the small end-to-end workload
def test_tiny_fp32_workload_end_to_end():
    """B=1, H=2, d=64, T=256 fp32: prefill, 16 decode steps, a 4-node chain verify, commit of 2."""
    W = wl.tiny_fp32()
    io = W.io
    q, k, v = W.prefill_inputs()
    w = W.weights()
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, io, chunk=W.chunk)
    st = ctx.new_state(W.B)
    o = ctx.la_prefill(dev(q, io), dev(k, io), dev(v, io), dev(w, "f32"), st)
    want, ost = orc.prefill_quadratic(q, k, v, w, W.phi, W.eps)
    assert rel_err(host(o), want) < TOL[io]
    for s in range(W.decode_steps):
        qs, ks, vs = W.decode_inputs(s)
        o = ctx.la_decode_step(dev(qs, io), dev(ks, io), dev(vs, io), dev(w, "f32"), st)
        want, ost = orc.decode_step(qs, ks, vs, w, W.phi, W.eps, ost)
        assert rel_err(host(o), want) < TOL[io]
    qd, kd, vd = W.draft_inputs(0)
    parent = np.stack([wl.chain_tree(W.tree_nodes)] * W.B)
    o = ctx.la_verify_tree(dev(qd, io), dev(kd, io), dev(vd, io), torch.from_numpy(parent).cuda(), dev(w, "f32"), st)
    assert rel_err(host(o), orc.verify_tree(qd, kd, vd, parent, w, W.phi, W.eps, ost)) < TOL[io]
    accept = np.full((W.B,), W.extra["accept_node"], dtype=np.int32)
    path, clen = ctx.la_commit(dev(kd, io), dev(vd, io), torch.from_numpy(parent).cuda(),
                               torch.from_numpy(accept).cuda(), st)
    ost, wpath, wlen = orc.commit(kd, vd, parent, accept, W.phi, ost, max_depth=ctx.max_depth)
    assert host(clen).tolist() == [2] and host(path)[0, :2].tolist() == [0, 1]
    np.testing.assert_array_equal(host(path), wpath)
    check_state(st, ost, TOL[io])
    assert int(st.pos[0]) == 256 + 16 + 2
