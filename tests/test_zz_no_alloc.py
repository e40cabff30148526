"""The allocation-free verification entry point against the float64 oracle and against the regular entry point.

Some users of the library run where device allocation is not allowed (a serving loop whose
memory pool owns the whole device, a plug-in that only receives a workspace and a stream), so
they cannot create a context.  la_verify_tree_noalloc serves them from a fixed array inside the
library.  This file is collected last on purpose: it runs after every other test, and it must
also pass alone in a fresh process.  Because the fixed array is shared by all calls and keeps
the previous call's contents, the check is made on two calls in a row, the first of which leaves
an error code behind that the second must not see.
"""
import numpy as np
import pytest
import torch

from oracle import la_oracle as orc
from paper_2406_07368_b200 import binding, workloads as wl
from tests._util import TOL, rel_err

pytestmark = pytest.mark.gpu


def _dev(x, io):
    return torch.from_numpy(np.ascontiguousarray(x)).to(binding.TORCH_DTYPE[io]).cuda()


def _host(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def _case(seed, io, B, H, d, N, W, zero_taps):
    q, k, v = wl.qkv(seed, (B, H, N, d), 0.7, io)
    w = wl.conv_weights(seed, H, d, W)
    if zero_taps:
        w = np.zeros_like(w)                               # the attention term alone
    parent = np.stack([wl.random_tree(wl.rng(seed, 4, 0, b), N, 5, 4) for b in range(B)]).astype(np.int32)
    return q, k, v, w, parent


@pytest.mark.parametrize("io,d,W,phi,eps", [("bf16", 128, 3, "elu1", 0.0), ("f32", 64, 5, "relu", 1e-6)])
def test_noalloc_verify_matches_oracle_and_regular_entry_point_twice(io, d, W, phi, eps):
    B, H, N = 5, 2, 33
    ctx = binding.Context(H, d, W, phi, eps, io, max_nodes=64, max_depth=64)
    # a committed state: the oracle's, after a short prompt, copied to the device
    q0, k0, v0 = wl.qkv(3, (B, H, 40, d), 0.5, io)
    _, ost = orc.prefill_quadratic(q0, k0, v0, wl.conv_weights(9, H, d, W), phi, eps)
    st = binding.State(torch.from_numpy(ost.S).float().cuda(), torch.from_numpy(ost.z).float().cuda(),
                       _dev(ost.win.astype(np.float32), io), torch.from_numpy(ost.pos).cuda())

    # first call: two malformed trees; second call: none, and zero taps -- it must not see the first call's codes
    for call, bad_seqs in ((0, (1, 3)), (1, ())):
        q, k, v, w, parent = _case(50 + call, io, B, H, d, N, W, zero_taps=call == 1)
        bad = parent.copy()
        for b in bad_seqs:
            bad[b, 4] = 7                                  # parent after child
        par = torch.from_numpy(bad).cuda()
        dq, dk, dv, dw = _dev(q, io), _dev(k, io), _dev(v, io), _dev(w, "f32")
        regular = torch.full((B, H, N, d), 55.0, dtype=binding.TORCH_DTYPE[io], device="cuda")
        got = regular.clone()
        seq_status = torch.full((B,), -1, dtype=torch.int32, device="cuda")
        before = st.clone()
        ctx.la_clear_device_status()
        ctx.la_verify_tree(dq, dk, dv, par, dw, st, out=regular)
        binding.la_verify_tree_noalloc(H, d, W, phi, eps, io, dq, dk, dv, par, dw, st, got, seq_status)
        torch.cuda.synchronize()
        good = [b for b in range(B) if b not in bad_seqs]
        want = orc.verify_tree(q[good], k[good], v[good], parent[good], w, phi, eps,
                               orc.State(ost.S[good], ost.z[good], ost.win[good], ost.pos[good]))
        assert rel_err(_host(got[good]), want) < TOL[io]                   # against the float64 oracle
        for i, b in enumerate(good):
            assert rel_err(_host(got[b]), want[i]) < TOL[io], b
        assert rel_err(_host(got[good]), _host(regular[good])) < TOL[io]   # and against the regular entry point
        expect = [binding.LA_ERR_BAD_TREE if b in bad_seqs else 0 for b in range(B)]
        for b in bad_seqs:
            assert torch.all(got[b] == 55.0)               # skipped sequences left unwritten
        assert ctx.la_last_device_status() == (binding.LA_ERR_BAD_TREE if bad_seqs else binding.LA_OK)
        assert seq_status.cpu().tolist() == expect
        for a, b in ((st.S, before.S), (st.z, before.z), (st.win, before.win), (st.pos, before.pos)):
            assert torch.equal(a, b)


def test_noalloc_rejects_batches_beyond_its_fixed_capacity():
    io, H, d, W, N = "bf16", 1, 64, 3, 2
    B = binding.LA_NOALLOC_MAX_SEQ + 1
    x = torch.zeros(B, H, N, d, dtype=torch.bfloat16, device="cuda")
    st = binding.State(torch.zeros(B, H, d, d, device="cuda"), torch.zeros(B, H, d, device="cuda"),
                       torch.zeros(B, H, W - 1, d, dtype=torch.bfloat16, device="cuda"),
                       torch.zeros(B, dtype=torch.int64, device="cuda"))
    par = torch.full((B, N), -1, dtype=torch.int32, device="cuda")
    w = torch.zeros(H, d, W, device="cuda")
    with pytest.raises(binding.LaError) as e:
        binding.la_verify_tree_noalloc(H, d, W, "elu1", 0.0, io, x, x, x, par, w, st, x.clone())
    assert e.value.code == binding.LA_ERR_TOO_LARGE and "LA_ERR_TOO_LARGE" in str(e.value)
    # the largest allowed batch goes through
    B = binding.LA_NOALLOC_MAX_SEQ
    out = torch.empty(B, H, N, d, dtype=torch.bfloat16, device="cuda")
    stat = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    binding.la_verify_tree_noalloc(H, d, W, "elu1", 0.0, io, x[:B].contiguous(), x[:B].contiguous(), x[:B].contiguous(),
                                   par[:B].contiguous(), w,
                                   binding.State(st.S[:B].contiguous(), st.z[:B].contiguous(), st.win[:B].contiguous(),
                                                 st.pos[:B].contiguous()), out, stat)
    torch.cuda.synchronize()
    assert int(stat.abs().sum()) == 0 and torch.isfinite(out.float()).all()
