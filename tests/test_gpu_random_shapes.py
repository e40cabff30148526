"""Seeded random shapes through every mode against the oracle: lengths, tap counts, tree sizes and feature maps that no
hand-picked case names."""
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


@pytest.mark.parametrize("case", range(12))
def test_random_shape_prefill_decode_verify_commit(case):
    g = wl.rng(9000, 1, case)
    io = "bf16" if case % 3 else "f32"
    d = 128 if (io == "bf16" and case % 2) else 64 if io == "f32" else (128 if case % 4 else 64)
    phi, eps = (("elu1", 0.0), ("relu", 1e-6))[int(g.integers(2))]
    B, H = int(g.integers(1, 4)), int(g.integers(1, 5))
    T, W, N = int(g.integers(1, 600)), int(g.integers(1, 33)), int(g.integers(1, 65))
    v_mean = float(g.integers(2))
    q, k, v = wl.qkv(9000 + case, (B, H, T, d), 0.6, io, v_mean=v_mean)
    w = wl.conv_weights(9000 + case, H, d, W)
    ctx = binding.Context(H, d, W, phi, eps, io, max_nodes=64, max_depth=64)
    st = ctx.new_state(B)
    T1 = int(g.integers(0, T))                               # prefill in two calls (the first may be empty)
    outs = []
    if T1:
        outs.append(ctx.la_prefill(dev(q[:, :, :T1], io), dev(k[:, :, :T1], io), dev(v[:, :, :T1], io), dev(w, "f32"), st))
    outs.append(ctx.la_prefill(dev(q[:, :, T1:], io), dev(k[:, :, T1:], io), dev(v[:, :, T1:], io), dev(w, "f32"), st,
                               init_state=T1 > 0))
    want, ost = orc.prefill_quadratic(q, k, v, w, phi, eps)
    assert rel_err(host(torch.cat(outs, dim=2)), want) < TOL[io]
    # a few decode steps
    for s in range(3):
        qs, ks, vs = wl.qkv(9100 + case, (B, H, d), 0.6, io, a=s, v_mean=v_mean)
        o = ctx.la_decode_step(dev(qs, io), dev(ks, io), dev(vs, io), dev(w, "f32"), st)
        wd, ost = orc.decode_step(qs, ks, vs, w, phi, eps, ost)
        assert rel_err(host(o), wd) < TOL[io]
    # a tree, verified and committed
    qd, kd, vd = wl.qkv(9200 + case, (B, H, N, d), 0.6, io, v_mean=v_mean)
    parent = np.stack([wl.random_tree(wl.rng(9300, 4, case, b), N, 8, 4) for b in range(B)]).astype(np.int32)
    accept = np.array([wl.random_accept(wl.rng(9300, 6, case, b), parent[b]) for b in range(B)], dtype=np.int32)
    par = torch.from_numpy(parent).cuda()
    before = st.clone()
    o = ctx.la_verify_tree(dev(qd, io), dev(kd, io), dev(vd, io), par, dev(w, "f32"), st)
    assert rel_err(host(o), orc.verify_tree(qd, kd, vd, parent, w, phi, eps, ost)) < TOL[io]
    assert torch.equal(st.S, before.S) and torch.equal(st.win, before.win)
    path, clen = ctx.la_commit(dev(kd, io), dev(vd, io), par, torch.from_numpy(accept).cuda(), st)
    ost, wpath, wlen = orc.commit(kd, vd, parent, accept, phi, ost, 64)
    np.testing.assert_array_equal(host(path), wpath)
    np.testing.assert_array_equal(host(clen), wlen)
    assert rel_err(host(st.S), ost.S) < TOL[io] and rel_err(host(st.z), ost.z) < TOL[io]
    np.testing.assert_array_equal(host(st.win), ost.win)
    np.testing.assert_array_equal(host(st.pos), ost.pos)
    assert ctx.la_last_device_status() == binding.LA_OK
