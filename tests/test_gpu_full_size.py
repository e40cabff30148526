"""Parity at the full workload sizes, in the launch configurations the benchmark times.

The whole batch runs on the GPU; the float64 oracle recomputes a sample of (sequence, head) units one by
one (every unit is independent of the others), plus the integer outputs of every sequence.
"""
import numpy as np
import pytest
import torch

from oracle import la_oracle as orc
from paper_2406_07368_b200 import binding, workloads as wl
from tests._util import TOL, rel_err

pytestmark = pytest.mark.gpu


def dev(x, io="bf16"):
    return torch.from_numpy(np.ascontiguousarray(x)).to(binding.TORCH_DTYPE[io]).cuda()


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def unit_state(st: binding.State, b, h):
    """Oracle state of one (sequence, head) unit taken from the device state."""
    return orc.State(host(st.S[b:b + 1, h:h + 1]), host(st.z[b:b + 1, h:h + 1]), host(st.win[b:b + 1, h:h + 1]),
                     st.pos[b:b + 1].cpu().numpy().copy())


def test_llama7b_prefill_full_size():
    W = wl.llama7b_prefill()
    q, k, v = W.prefill_inputs()
    w = W.weights()
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, W.io, chunk=W.chunk)
    st = ctx.new_state(W.B)
    o = ctx.la_prefill(dev(q), dev(k), dev(v), dev(w, "f32"), st)
    assert ctx.la_last_device_status() == binding.LA_OK
    for b, h in ((0, 0), (1, 17), (3, 31)):
        sl = (slice(b, b + 1), slice(h, h + 1))
        want, wst = orc.prefill_quadratic(q[sl], k[sl], v[sl], w[h:h + 1], W.phi, W.eps)
        assert rel_err(host(o[sl]), want) < TOL["bf16"]
        assert rel_err(host(st.S[sl]), wst.S) < TOL["bf16"]
        assert rel_err(host(st.z[sl]), wst.z) < TOL["bf16"]
        np.testing.assert_array_equal(host(st.win[sl]), wst.win)
    assert st.pos.tolist() == [W.T] * W.B


def test_long_prefill_full_size_then_decode():
    W = wl.long_prefill()
    q, k, v = W.prefill_inputs()
    w = W.weights()
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, W.io, chunk=W.chunk)
    ws = torch.empty(ctx.la_prefill_workspace_bytes(W.B, W.T), dtype=torch.uint8, device="cuda")
    assert ws.numel() > 0                       # 32 chains: the sequence-split path, as in the benchmark
    ctx.la_set_workspace(ws)
    st = ctx.new_state(W.B)
    o = ctx.la_prefill(dev(q), dev(k), dev(v), dev(w, "f32"), st)
    heads = (0, 13, 31)
    ost = {}
    for h in heads:
        sl = (slice(0, 1), slice(h, h + 1))
        want, ost[h] = orc.prefill_chunked(q[sl], k[sl], v[sl], w[h:h + 1], W.phi, W.eps, 256)
        assert rel_err(host(o[sl]), want) < TOL["bf16"]
        assert rel_err(host(st.S[sl]), ost[h].S) < TOL["bf16"]
        assert rel_err(host(st.z[sl]), ost[h].z) < TOL["bf16"]
        np.testing.assert_array_equal(host(st.win[sl]), ost[h].win)
    # the decode tail: oracle continues from its own state, the GPU from its own
    for s in range(64):
        qs, ks, vs = W.decode_inputs(s)
        od = ctx.la_decode_step(dev(qs), dev(ks), dev(vs), dev(w, "f32"), st)
        for h in heads:
            want, ost[h] = orc.decode_step(qs[:, h:h + 1], ks[:, h:h + 1], vs[:, h:h + 1], w[h:h + 1], W.phi, W.eps, ost[h])
            assert rel_err(host(od[:, h:h + 1]), want) < TOL["bf16"], (s, h)
    assert int(st.pos[0]) == W.T + 64
    assert ctx.la_last_device_status() == binding.LA_OK


def test_batched_decode_full_batch():
    """64 sequences x 32 heads: prompt of 2048 tokens, then decode steps at the full batch size."""
    W = wl.batched_decode()
    gen = torch.Generator(device="cuda").manual_seed(W.seed)
    shape = (W.B, W.H, W.T, W.d)
    q, k, v = (torch.randn(shape, generator=gen, device="cuda", dtype=torch.float32).bfloat16() for _ in range(3))
    w = W.weights()
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, W.io)
    st = ctx.new_state(W.B)
    ctx.la_prefill(q, k, v, dev(w, "f32"), st)
    units = ((0, 0), (21, 7), (63, 31))
    ost = {}
    for b, h in units:
        sl = (slice(b, b + 1), slice(h, h + 1))
        _, ost[(b, h)] = orc.prefill_chunked(host(q[sl]), host(k[sl]), host(v[sl]), w[h:h + 1], W.phi, W.eps, 256)
        assert rel_err(host(st.S[sl]), ost[(b, h)].S) < TOL["bf16"]
    del q, k, v
    steps = 96
    for s in range(steps):
        qs, ks, vs = W.decode_inputs(s)
        od = ctx.la_decode_step(dev(qs), dev(ks), dev(vs), dev(w, "f32"), st)
        for b, h in units:
            sl = (slice(b, b + 1), slice(h, h + 1))
            want, ost[(b, h)] = orc.decode_step(qs[sl], ks[sl], vs[sl], w[h:h + 1], W.phi, W.eps, ost[(b, h)])
            assert rel_err(host(od[sl]), want) < TOL["bf16"], (s, b, h)
    for b, h in units:
        sl = (slice(b, b + 1), slice(h, h + 1))
        assert rel_err(host(st.S[sl]), ost[(b, h)].S) < TOL["bf16"]
        np.testing.assert_array_equal(host(st.win[sl]), ost[(b, h)].win)
    assert st.pos.tolist() == [W.T + steps] * W.B
    assert ctx.la_last_device_status() == binding.LA_OK


def test_tree_verify_full_size_rounds():
    """16 sequences, 1024-token prompt, 64-node trees: rounds of verify + commit with the state carried."""
    W = wl.tree_verify()
    q, k, v = W.prefill_inputs()
    w = W.weights()
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, W.io, max_nodes=W.tree_nodes, max_depth=W.max_depth)
    st = ctx.new_state(W.B)
    ctx.la_prefill(dev(q), dev(k), dev(v), dev(w, "f32"), st)
    units = ((0, 0), (7, 19), (15, 31))
    ost = {}
    for b, h in units:
        sl = (slice(b, b + 1), slice(h, h + 1))
        _, ost[(b, h)] = orc.prefill_chunked(q[sl], k[sl], v[sl], w[h:h + 1], W.phi, W.eps, 256)
    for rnd in range(8):
        qd, kd, vd = W.draft_inputs(rnd)
        parent, accept = W.trees(rnd)
        par, acc = torch.from_numpy(parent).cuda(), torch.from_numpy(accept).cuda()
        before = st.clone()
        o = ctx.la_verify_tree(dev(qd), dev(kd), dev(vd), par, dev(w, "f32"), st)
        assert torch.equal(st.S, before.S) and torch.equal(st.z, before.z) and torch.equal(st.win, before.win)
        path, clen = ctx.la_commit(dev(kd), dev(vd), par, acc, st)
        # integer outputs of every sequence against a parent walk done here
        for b in range(W.B):
            chain, m = [], int(accept[b])
            while m >= 0:
                chain.append(m)
                m = int(parent[b, m])
            chain.reverse()
            assert int(clen[b]) == len(chain)
            assert path[b].tolist() == chain + [-1] * (W.max_depth - len(chain))
        for b, h in units:
            sl = (slice(b, b + 1), slice(h, h + 1))
            want = orc.verify_tree(qd[sl], kd[sl], vd[sl], parent[b:b + 1], w[h:h + 1], W.phi, W.eps, ost[(b, h)])
            assert rel_err(host(o[sl]), want) < TOL["bf16"], (rnd, b, h)
            ost[(b, h)], _, _ = orc.commit(kd[sl], vd[sl], parent[b:b + 1], accept[b:b + 1], W.phi, ost[(b, h)],
                                           W.max_depth)
    for b, h in units:
        sl = (slice(b, b + 1), slice(h, h + 1))
        assert rel_err(host(st.S[sl]), ost[(b, h)].S) < TOL["bf16"]
        assert rel_err(host(st.z[sl]), ost[(b, h)].z) < TOL["bf16"]
        np.testing.assert_array_equal(host(st.win[sl]), ost[(b, h)].win)
        assert int(st.pos[b]) == int(ost[(b, h)].pos[0])
    assert ctx.la_last_device_status() == binding.LA_OK


def test_prompt_gen_pairs_prefill_then_generate():
    """The two shorter (prompt, generation) pairs end to end at full head count: every output token and the final
    state against the oracle's quadratic definition over the whole P + G sequence."""
    W = wl.prompt_gen()
    w = W.weights()
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, W.io, chunk=W.chunk)
    for i, (P, G) in enumerate(W.extra["shapes"]):
        if P + G > 600:
            continue
        q, k, v = wl.qkv(W.seed + i, (W.B, W.H, P + G, W.d), W.scale, W.io)
        st = ctx.new_state(W.B)
        op = ctx.la_prefill(dev(q[:, :, :P]), dev(k[:, :, :P]), dev(v[:, :, :P]), dev(w, "f32"), st)
        og = [ctx.la_decode_step(dev(q[:, :, P + g]), dev(k[:, :, P + g]), dev(v[:, :, P + g]), dev(w, "f32"), st)
              for g in range(G)]
        want, wst = orc.prefill_quadratic(q, k, v, w, W.phi, W.eps)
        assert rel_err(host(op), want[:, :, :P]) < TOL["bf16"], (P, G)
        assert rel_err(np.stack([host(o) for o in og], axis=2), want[:, :, P:]) < TOL["bf16"], (P, G)
        assert rel_err(host(st.S), wst.S) < TOL["bf16"] and rel_err(host(st.z), wst.z) < TOL["bf16"]
        np.testing.assert_array_equal(host(st.win), wst.win)
        assert int(st.pos[0]) == P + G
    assert ctx.la_last_device_status() == binding.LA_OK
