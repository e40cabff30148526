"""The pieces of the sequence-parallel prefill on the GPU: la_segment_state and la_state_prefix against the oracle,
and the whole exchange with the ranks played one after the other on one GPU (their kernels do not wait on one
another: phase 1 of every rank, the gather by stacking, phase 2 of every rank)."""
import numpy as np
import pytest
import torch

from oracle import la_oracle as orc
from paper_2406_07368_b200 import binding, seqpar, workloads as wl
from tests._util import TOL, rel_err

pytestmark = pytest.mark.gpu


def dev(x, io):
    return torch.from_numpy(np.ascontiguousarray(x)).to(binding.TORCH_DTYPE[io]).cuda()


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64) if t.is_floating_point() else t.cpu().numpy()


@pytest.mark.parametrize("kernel", [0, 1])
@pytest.mark.parametrize("io,d,phi,T", [("bf16", 128, "elu1", 700), ("bf16", 128, "relu", 129), ("bf16", 64, "elu1", 100),
                                        ("f32", 64, "elu1", 257), ("f32", 128, "relu", 33), ("bf16", 128, "elu1", 1)])
def test_segment_state_matches_oracle(kernel, io, d, phi, T):
    B, H = 2, 3
    _, k, v = wl.qkv(4000 + T, (B, H, T, d), 0.5, io, v_mean=0.5)
    ctx = binding.Context(H, d, 3, phi, 0.0, io)
    ctx.la_set_prefill_kernel(kernel)
    dS, dz = ctx.la_segment_state(dev(k, io), dev(v, io))
    assert ctx.la_last_device_status() == binding.LA_OK
    _, st = orc.prefill_quadratic(np.zeros_like(k), k, v, np.zeros((H, d, 3)), phi, 1.0)     # (only the state is used)
    assert rel_err(host(dS), st.S) < TOL[io] and rel_err(host(dz), st.z) < TOL[io]


def test_state_prefix_adds_the_parts_before_a_rank():
    B, H, d, n = 2, 3, 64, 5
    ctx = binding.Context(H, d, 3, "elu1", 0.0, "f32")
    g = torch.Generator(device="cuda").manual_seed(1)
    dS = torch.randn(n, B, H, d, d, device="cuda", generator=g)
    dz = torch.randn(n, B, H, d, device="cuda", generator=g)
    S0, z0 = torch.randn(B, H, d, d, device="cuda", generator=g), torch.randn(B, H, d, device="cuda", generator=g)
    for count in (0, 1, 3, 5):
        S, z = ctx.la_state_prefix(dS, dz, count, S0, z0)
        np.testing.assert_allclose(host(S), host(S0) + host(dS[:count]).sum(0), rtol=1e-5, atol=1e-5)
        np.testing.assert_allclose(host(z), host(z0) + host(dz[:count]).sum(0), rtol=1e-5, atol=1e-5)
        S, z = ctx.la_state_prefix(dS, dz, count)
        np.testing.assert_allclose(host(S), host(dS[:count]).sum(0), rtol=1e-5, atol=1e-5)


@pytest.mark.parametrize("io,d,phi,eps,W,T,world,with_state", [
    ("bf16", 128, "elu1", 0.0, 3, 1000, 2, False), ("bf16", 128, "relu", 1e-6, 5, 4099, 4, True),
    ("bf16", 128, "elu1", 0.0, 32, 700, 3, False), ("f32", 64, "elu1", 0.0, 4, 300, 2, True),
    ("bf16", 128, "elu1", 0.0, 3, 100, 4, False)])          # fewer tokens than ranks x 128: empty stretches
def test_sequence_parallel_prefill_equals_the_whole_sequence(io, d, phi, eps, W, T, world, with_state):
    B, H = 1, 2
    q, k, v = wl.qkv(4100 + T, (B, H, T, d), d ** -0.5 if io == "bf16" else 1.0, io, v_mean=0.5)
    w = wl.conv_weights(T, H, d, W)
    ctx = binding.Context(H, d, W, phi, eps, io)
    ops = seqpar.BindingOps(ctx)
    state0 = ost0 = None
    if with_state:
        q0, k0, v0 = wl.qkv(4101, (B, H, 70, d), 0.5, io)
        _, ost0 = orc.prefill_quadratic(q0, k0, v0, w, phi, eps)
        state0 = (torch.from_numpy(ost0.S).float().cuda(), torch.from_numpy(ost0.z).float().cuda(),
                  dev(ost0.win.astype(np.float32), io), torch.from_numpy(ost0.pos).cuda())
    dq, dk, dv, dw = dev(q, io), dev(k, io), dev(v, io), dev(w, "f32")
    cuts = [seqpar.token_shard(T, r, world) for r in range(world)]
    parts = [seqpar.local_partial(ops, dk[:, :, lo:hi], dv[:, :, lo:hi], W) for lo, hi in cuts]
    dS_all, dz_all = torch.stack([p.dS for p in parts]), torch.stack([p.dz for p in parts])
    tails, counts = torch.stack([p.tail for p in parts]), [p.count for p in parts]
    want, wst = orc.prefill_quadratic(q, k, v, w, phi, eps, ost0)
    outs = []
    for r, (lo, hi) in enumerate(cuts):
        o, S, z, win, pos = seqpar.finish_rank(ops, r, dq[:, :, lo:hi], dk[:, :, lo:hi], dv[:, :, lo:hi], dw, dS_all,
                                               dz_all, tails, counts, state0)
        if o is not None:
            outs.append(o)
            assert rel_err(host(o), want[:, :, lo:hi]) < TOL[io], r      # every stretch on its own
        assert rel_err(host(S), wst.S) < TOL[io] and rel_err(host(z), wst.z) < TOL[io]
        np.testing.assert_array_equal(host(win), wst.win)
        np.testing.assert_array_equal(host(pos), wst.pos)
    assert rel_err(host(torch.cat(outs, dim=2)), want) < TOL[io]
    assert ctx.la_last_device_status() == binding.LA_OK
