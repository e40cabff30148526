"""Out-of-bounds and repeatability checks on the GPU: every output and state buffer sits between guard words that must
survive the calls, and a call repeated on the same inputs gives the same bits."""
import numpy as np
import pytest
import torch

from paper_2406_07368_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu

GUARD = 4096          # bytes on either side of every carved tensor
PATTERN = 0xA5


class Arena:
    """One byte buffer filled with a pattern; tensors are carved out of it with guard bytes around each."""

    def __init__(self, nbytes):
        self.buf = torch.full((nbytes,), PATTERN, dtype=torch.uint8, device="cuda")
        self.off = 0
        self.used = []

    def take(self, shape, dtype, fill=None):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        start = (self.off + GUARD + 255) // 256 * 256
        t = self.buf[start:start + n].view(dtype).view(*shape)
        if fill is not None:
            t.fill_(fill)
        self.used.append((start, start + n))
        self.off = start + n
        assert self.off + GUARD <= self.buf.numel()
        return t

    def check(self):
        mask = torch.ones(self.buf.numel(), dtype=torch.bool, device="cuda")
        for a, b in self.used:
            mask[a:b] = False
        assert bool((self.buf[mask] == PATTERN).all()), "a kernel wrote outside its buffers"


def dev(x, io="bf16"):
    return torch.from_numpy(np.ascontiguousarray(x)).to(binding.TORCH_DTYPE[io]).cuda()


@pytest.mark.parametrize("T,W", [(1, 3), (127, 3), (300, 4), (333, 32)])
def test_guards_survive_prefill_decode_verify_commit(T, W):
    io, B, H, d, N = "bf16", 2, 3, 128, 37
    q, k, v = wl.qkv(T + W, (B, H, T, d), d ** -0.5, io)
    w = dev(wl.conv_weights(1, H, d, W), "f32")
    ctx = binding.Context(H, d, W, "elu1", 0.0, io, max_nodes=64, max_depth=8)
    ar = Arena(64 << 20)
    st = binding.State(ar.take((B, H, d, d), torch.float32, 0.0), ar.take((B, H, d), torch.float32, 0.0),
                       ar.take((B, H, W - 1, d), torch.bfloat16, 0.0), ar.take((B,), torch.int64, 0))
    o = ar.take((B, H, T, d), torch.bfloat16)
    ctx.la_prefill(dev(q), dev(k), dev(v), w, st, out=o)
    od = ar.take((B, H, d), torch.bfloat16)
    qs, ks, vs = wl.qkv(9, (B, H, d), 0.7, io)
    ctx.la_decode_step(dev(qs), dev(ks), dev(vs), w, st, out=od)
    qd, kd, vd = wl.qkv(10, (B, H, N, d), 0.7, io)
    parent, accept = wl.tree_batch(3, 0, B, N, max_depth=6)
    ov = ar.take((B, H, N, d), torch.bfloat16)
    par = torch.from_numpy(parent).cuda()
    ctx.la_verify_tree(dev(qd), dev(kd), dev(vd), par, w, st, out=ov)
    draft, pred_root, pred = wl.token_batch(3, 0, B, N, vocab=2)
    node, length, nxt = (ar.take((B,), torch.int32) for _ in range(3))
    ctx.la_accept_greedy(par, *(torch.from_numpy(x).cuda() for x in (draft, pred_root, pred)), accept_node=node,
                         accept_len=length, next_token=nxt)
    path, clen = ar.take((B, 8), torch.int32), ar.take((B,), torch.int32)
    ctx.la_commit(dev(kd), dev(vd), par, torch.from_numpy(accept).cuda(), st, path_out=path, commit_len=clen)
    torch.cuda.synchronize()
    assert ctx.la_last_device_status() == binding.LA_OK
    ar.check()
    assert torch.isfinite(o.float()).all() and torch.isfinite(ov.float()).all() and torch.isfinite(st.S).all()


def test_repeated_calls_give_the_same_bits():
    io, B, H, d, T, W, N = "bf16", 3, 4, 128, 700, 3, 64
    q, k, v = (dev(x) for x in wl.qkv(5, (B, H, T, d), d ** -0.5, io))
    qd, kd, vd = (dev(x) for x in wl.qkv(6, (B, H, N, d), 0.7, io))
    w = dev(wl.conv_weights(2, H, d, W), "f32")
    parent, accept = wl.tree_batch(4, 0, B, N)
    par, acc = torch.from_numpy(parent).cuda(), torch.from_numpy(accept).cuda()
    ctx = binding.Context(H, d, W, "elu1", 0.0, io, max_nodes=64, max_depth=5)
    results = []
    for _ in range(2):
        st = ctx.new_state(B)
        o = ctx.la_prefill(q, k, v, w, st)
        ov = ctx.la_verify_tree(qd, kd, vd, par, w, st)
        path, clen = ctx.la_commit(kd, vd, par, acc, st)
        od = ctx.la_decode_step(qd[:, :, 0].contiguous(), kd[:, :, 0].contiguous(), vd[:, :, 0].contiguous(), w, st)
        results.append((o, ov, od, path, clen, st.S.clone(), st.z.clone(), st.win.clone(), st.pos.clone()))
    for a, b in zip(*results):
        assert torch.equal(a, b)


def test_a_wait_that_nobody_ends_runs_out_and_reports_it():
    """The bounded wait of the kernels, on a barrier nobody arrives on: it gives up after the limit, the status word
    says so, and the context keeps working."""
    ctx = binding.Context(2, 128, 3, "elu1", 0.0, "bf16")
    assert ctx.la_last_device_status() == binding.LA_OK
    waited = ctx.la_selftest_wait_timeout(20000)                     # 20 ms
    assert ctx.la_last_device_status() == binding.LA_ERR_TIMEOUT
    assert 20e6 <= waited < 200e6                                    # at least the limit, and not much more
    ctx.la_clear_device_status()
    assert ctx.la_last_device_status() == binding.LA_OK
    st = ctx.new_state(1)
    x = torch.randn(1, 2, 130, 128, device="cuda").bfloat16() * 0.1
    o = ctx.la_prefill(x, x, x, torch.ones(2, 128, 3, device="cuda"), st)
    assert ctx.la_last_device_status() == binding.LA_OK and torch.isfinite(o.float()).all()


@pytest.mark.parametrize("io,d,T,W,C", [("bf16", 128, 333, 5, 64), ("f32", 64, 200, 32, 37), ("bf16", 64, 300, 3, 256)])
def test_guards_survive_the_three_branch_block_and_the_segment_sums(io, d, T, W, C):
    B, H = 2, 3
    dt = binding.TORCH_DTYPE[io]
    q, k, v = (dev(x, io) for x in wl.qkv(T + W + C, (B, H, T, d), 0.5, io))
    w = dev(wl.conv_weights(2, H, d, W), "f32")
    ctx = binding.Context(H, d, W, "elu1", 0.0, io)
    ar = Arena(64 << 20)
    st = binding.State(ar.take((B, H, d, d), torch.float32, 0.0), ar.take((B, H, d), torch.float32, 0.0),
                       ar.take((B, H, W - 1, d), dt, 0.0), ar.take((B,), torch.int64, 0))
    o = ar.take((B, H, T, d), dt)
    ctx.la_prefill_grouped(q, k, v, w, st, C, 0.7, d ** -0.5, out=o)
    dS, dz = ar.take((B, H, d, d), torch.float32), ar.take((B, H, d), torch.float32)
    ctx.la_segment_state(k, v, dS=dS, dz=dz)
    parts_S, parts_z = torch.stack([dS, dS, dS]), torch.stack([dz, dz, dz])
    S2, z2 = ctx.la_state_prefix(parts_S, parts_z, 2, st.S, st.z)
    torch.cuda.synchronize()
    assert ctx.la_last_device_status() == binding.LA_OK
    ar.check()
    assert torch.isfinite(o.float()).all() and torch.isfinite(dS).all() and torch.isfinite(S2).all()
    assert torch.allclose(S2, st.S + 2 * dS, rtol=1e-5, atol=1e-5) and torch.allclose(z2, st.z + 2 * dz, rtol=1e-5, atol=1e-5)
    assert st.pos.tolist() == [T] * B


def test_two_contexts_on_two_streams_do_not_disturb_each_other():
    """Calls of two contexts issued on two streams, interleaved, give the bits of the same calls issued alone."""
    io, B, H, d, T, W = "bf16", 2, 4, 128, 700, 3
    q, k, v = (dev(x, io) for x in wl.qkv(77, (B, H, T, d), d ** -0.5, io))
    w = dev(wl.conv_weights(3, H, d, W), "f32")
    ca, cb = binding.Context(H, d, W, "elu1", 0.0, io), binding.Context(H, d, W, "relu", 1e-6, io)
    ref = []
    for c in (ca, cb):
        st = c.new_state(B)
        ref.append((c.la_prefill(q, k, v, w, st), st))
    torch.cuda.synchronize()
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    outs = []
    for _ in range(3):
        got = []
        for c, s in ((ca, sa), (cb, sb)):
            st = c.new_state(B)
            with torch.cuda.stream(s):
                got.append((c.la_prefill(q, k, v, w, st, stream=s), st))
        outs.append(got)
    torch.cuda.synchronize()
    for got in outs:
        for (o, st), (ro, rst) in zip(got, ref):
            assert torch.equal(o, ro) and torch.equal(st.S, rst.S) and torch.equal(st.z, rst.z)
    assert ca.la_last_device_status() == binding.LA_OK and cb.la_last_device_status() == binding.LA_OK
