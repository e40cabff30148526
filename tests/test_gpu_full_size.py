"""Parity at the full workload sizes, in the launch configurations the benchmark times.

The whole batch runs on the GPU; the float64 oracle recomputes a sample of (sequence, head) units one by
one (every unit is independent of the others), plus the integer outputs of every sequence.
"""
import numpy as np
import pytest
import torch

from oracle import la_oracle as orc
from paper_2406_07368_b200 import binding, workloads as wl
from tests._util import TOL, rel_err, rel_err_octaves

pytestmark = pytest.mark.gpu


def dev(x, io="bf16"):
    return torch.from_numpy(np.ascontiguousarray(x)).to(binding.TORCH_DTYPE[io]).cuda()


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def unit_state(st: binding.State, b, h):
    """Oracle state of one (sequence, head) unit taken from the device state."""
    return orc.State(host(st.S[b:b + 1, h:h + 1]), host(st.z[b:b + 1, h:h + 1]), host(st.win[b:b + 1, h:h + 1]),
                     st.pos[b:b + 1].cpu().numpy().copy())


def sampled_units(B, H, n):
    """n (sequence, head) pairs spread over the batch, the first and the last unit among them."""
    units = [(0, 0), (B - 1, H - 1)]
    i = 0
    while len(units) < min(n, B * H):
        u = ((3 * i + 1) % B, (7 * i + 5) % H)
        if u not in units:
            units.append(u)
        i += 1
    return units


def zero_taps(w):
    """The same layer with the convolution branch switched off: the output is the attention term alone."""
    return np.zeros_like(w)


def test_llama7b_prefill_full_size():
    W = wl.llama7b_prefill()
    q, k, v = W.prefill_inputs()
    w = W.weights()
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, W.io, chunk=W.chunk)
    st = ctx.new_state(W.B)
    dq, dk, dv = dev(q), dev(k), dev(v)
    o = ctx.la_prefill(dq, dk, dv, dev(w, "f32"), st)
    st0 = ctx.new_state(W.B)
    o0 = ctx.la_prefill(dq, dk, dv, dev(zero_taps(w), "f32"), st0)         # attention term alone, same launch shape
    assert ctx.la_last_device_status() == binding.LA_OK
    for i, (b, h) in enumerate(sampled_units(W.B, W.H, 16)):
        sl = (slice(b, b + 1), slice(h, h + 1))
        want, wst = orc.prefill_quadratic(q[sl], k[sl], v[sl], w[h:h + 1], W.phi, W.eps)
        assert rel_err(host(o[sl]), want) < TOL["bf16"], (b, h)
        assert rel_err(host(st.S[sl]), wst.S) < TOL["bf16"]
        assert rel_err(host(st.z[sl]), wst.z) < TOL["bf16"]
        np.testing.assert_array_equal(host(st.win[sl]), wst.win)
        if i < 8:
            la = want - orc.causal_dwconv(v[sl].astype(np.float64), w[h:h + 1].astype(np.float64),
                                          np.zeros((1, 1, W.W - 1, W.d)))
            assert rel_err_octaves(host(o0[sl]), la) < TOL["bf16"], (b, h)   # octave by octave: see tests/_util.py
            assert rel_err(host(o0[sl])[:, :, -128:], la[:, :, -128:]) < TOL["bf16"], (b, h)
    assert torch.equal(st.S, st0.S) and torch.equal(st.z, st0.z)            # the state does not depend on the taps
    assert st.pos.tolist() == [W.T] * W.B


def test_prefill_taps32_full_size():
    """The 32-tap prefill of the bench line (long-window epilogue), full batch, sampled units against the definition."""
    W = wl.prefill_taps32()
    q, k, v = W.prefill_inputs()
    w = W.weights()
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, W.io, chunk=W.chunk)
    st = ctx.new_state(W.B)
    o = ctx.la_prefill(dev(q), dev(k), dev(v), dev(w, "f32"), st)
    assert ctx.la_last_device_status() == binding.LA_OK
    for b, h in sampled_units(W.B, W.H, 8):
        sl = (slice(b, b + 1), slice(h, h + 1))
        want, wst = orc.prefill_quadratic(q[sl], k[sl], v[sl], w[h:h + 1], W.phi, W.eps)
        assert rel_err(host(o[sl]), want) < TOL["bf16"], (b, h)
        assert rel_err(host(o[sl])[:, :, -128:], want[:, :, -128:]) < TOL["bf16"], (b, h)
        assert rel_err(host(st.S[sl]), wst.S) < TOL["bf16"] and rel_err(host(st.z[sl]), wst.z) < TOL["bf16"]
        np.testing.assert_array_equal(host(st.win[sl]), wst.win)
    assert st.pos.tolist() == [W.T] * W.B


def test_grouped_block_full_size():
    """The three-branch block of the bench line (groups of 64 on the tensor cores), full batch, sampled units."""
    W = wl.grouped_block()
    q, k, v = W.prefill_inputs()
    w = W.weights()
    alpha, scale = W.extra["alpha"], W.extra["softmax_scale"]
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, W.io, chunk=W.chunk)
    st = ctx.new_state(W.B)
    o = ctx.la_prefill_grouped(dev(q), dev(k), dev(v), dev(w, "f32"), st, W.chunk, alpha, scale)
    assert ctx.la_last_device_status() == binding.LA_OK
    for b, h in sampled_units(W.B, W.H, 6):
        sl = (slice(b, b + 1), slice(h, h + 1))
        want, wst = orc.prefill_grouped_block(q[sl], k[sl], v[sl], w[h:h + 1], W.phi, W.eps, W.chunk, alpha, scale)
        assert rel_err(host(o[sl]), want) < TOL["bf16"], (b, h)
        assert rel_err(host(o[sl])[:, :, -128:], want[:, :, -128:]) < TOL["bf16"], (b, h)
        assert rel_err(host(st.S[sl]), wst.S) < TOL["bf16"] and rel_err(host(st.z[sl]), wst.z) < TOL["bf16"]
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
    dq, dk, dv = dev(q), dev(k), dev(v)
    o = ctx.la_prefill(dq, dk, dv, dev(w, "f32"), st)
    st0 = ctx.new_state(W.B)
    o0 = ctx.la_prefill(dq, dk, dv, dev(zero_taps(w), "f32"), st0)         # attention term alone
    heads = (0, 5, 13, 22, 31)
    ost = {}
    for h in heads:
        sl = (slice(0, 1), slice(h, h + 1))
        want, ost[h] = orc.prefill_chunked(q[sl], k[sl], v[sl], w[h:h + 1], W.phi, W.eps, 256)
        assert rel_err(host(o[sl]), want) < TOL["bf16"]
        assert rel_err(host(st.S[sl]), ost[h].S) < TOL["bf16"]
        assert rel_err(host(st.z[sl]), ost[h].z) < TOL["bf16"]
        np.testing.assert_array_equal(host(st.win[sl]), ost[h].win)
        la, _ = orc.prefill_chunked(q[sl], k[sl], v[sl], zero_taps(w[h:h + 1]), W.phi, W.eps, 256)
        got0 = host(o0[sl])
        assert rel_err_octaves(got0, la) < TOL["bf16"], h                   # octave by octave: see tests/_util.py
        for lo in range(4096, W.T, 4096):                                    # and stretch by stretch along the sequence
            assert rel_err(got0[:, :, lo:lo + 4096], la[:, :, lo:lo + 4096]) < TOL["bf16"], (h, lo)
    # the decode tail: oracle continues from its own state, the GPU from its own
    for s in range(W.decode_steps):
        qs, ks, vs = W.decode_inputs(s)
        od = ctx.la_decode_step(dev(qs), dev(ks), dev(vs), dev(w, "f32"), st)
        for h in heads[:3]:
            want, ost[h] = orc.decode_step(qs[:, h:h + 1], ks[:, h:h + 1], vs[:, h:h + 1], w[h:h + 1], W.phi, W.eps, ost[h])
            assert rel_err(host(od[:, h:h + 1]), want) < TOL["bf16"], (s, h)
    for h in heads[:3]:
        sl = (slice(0, 1), slice(h, h + 1))
        assert rel_err(host(st.S[sl]), ost[h].S) < TOL["bf16"] and rel_err(host(st.z[sl]), ost[h].z) < TOL["bf16"]
        np.testing.assert_array_equal(host(st.win[sl]), ost[h].win)
    assert int(st.pos[0]) == W.T + W.decode_steps == 32768 + 512
    assert ctx.la_last_device_status() == binding.LA_OK


def test_batched_decode_full_batch():
    """64 sequences x 32 heads: the seeded prompt of 2048 tokens, then all 1024 decode steps at the full batch size.
    A second state set runs the same steps with zero taps, so that the attention term is compared on its own."""
    W = wl.batched_decode()
    w = W.weights()
    w0 = zero_taps(w)
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, W.io)
    shape = (W.B, W.H, W.T, W.d)
    q, k, v = (torch.empty(shape, dtype=torch.bfloat16, device="cuda") for _ in range(3))
    units = ((0, 0), (21, 7), (63, 31))
    host_prompt = {}
    for b in range(W.B):                                   # the prompt is drawn sequence by sequence (6 GB as one array)
        qb, kb, vb = W.prompt_of_sequence(b)
        q[b:b + 1], k[b:b + 1], v[b:b + 1] = dev(qb), dev(kb), dev(vb)
        for ub, h in units:
            if ub == b:
                host_prompt[(ub, h)] = tuple(x[:, h:h + 1].copy() for x in (qb, kb, vb))
    st = ctx.new_state(W.B)
    ctx.la_prefill(q, k, v, dev(w, "f32"), st)
    ost, ost0 = {}, {}
    for (b, h), (qu, ku, vu) in host_prompt.items():
        sl = (slice(b, b + 1), slice(h, h + 1))
        _, ost[(b, h)] = orc.prefill_chunked(qu, ku, vu, w[h:h + 1], W.phi, W.eps, 256)
        assert rel_err(host(st.S[sl]), ost[(b, h)].S) < TOL["bf16"]
        ost0[(b, h)] = ost[(b, h)].copy()
    del q, k, v
    st0 = st.clone()
    dw, dw0 = dev(w, "f32"), dev(w0, "f32")
    steps = W.decode_steps
    assert steps == 1024
    for s in range(steps):
        qs, ks, vs = W.decode_inputs(s)
        dq, dk, dv = dev(qs), dev(ks), dev(vs)
        od = ctx.la_decode_step(dq, dk, dv, dw, st)
        od0 = ctx.la_decode_step(dq, dk, dv, dw0, st0)
        for b, h in units:
            sl = (slice(b, b + 1), slice(h, h + 1))
            want, ost[(b, h)] = orc.decode_step(qs[sl], ks[sl], vs[sl], w[h:h + 1], W.phi, W.eps, ost[(b, h)])
            assert rel_err(host(od[sl]), want) < TOL["bf16"], (s, b, h)
            la, ost0[(b, h)] = orc.decode_step(qs[sl], ks[sl], vs[sl], w0[h:h + 1], W.phi, W.eps, ost0[(b, h)])
            assert rel_err(host(od0[sl]), la) < TOL["bf16"], (s, b, h)
    for b, h in units:
        sl = (slice(b, b + 1), slice(h, h + 1))
        assert rel_err(host(st.S[sl]), ost[(b, h)].S) < TOL["bf16"]
        assert rel_err(host(st.z[sl]), ost[(b, h)].z) < TOL["bf16"]
        np.testing.assert_array_equal(host(st.win[sl]), ost[(b, h)].win)
    assert torch.equal(st.S, st0.S) and torch.equal(st.win, st0.win)
    assert st.pos.tolist() == [W.T + steps] * W.B
    assert ctx.la_last_device_status() == binding.LA_OK


def test_tree_verify_full_size_rounds():
    """16 sequences, 1024-token prompt, 64-node trees: all 256 rounds of verify + commit with the state carried, and
    the state after the last round compared.  Every round is also verified with zero taps (attention term alone)."""
    W = wl.tree_verify()
    q, k, v = W.prefill_inputs()
    w = W.weights()
    w0 = zero_taps(w)
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, W.io, max_nodes=W.tree_nodes, max_depth=W.max_depth)
    st = ctx.new_state(W.B)
    dw, dw0 = dev(w, "f32"), dev(w0, "f32")
    ctx.la_prefill(dev(q), dev(k), dev(v), dw, st)
    units = ((0, 0), (7, 19), (15, 31))
    ost = {}
    for b, h in units:
        sl = (slice(b, b + 1), slice(h, h + 1))
        _, ost[(b, h)] = orc.prefill_chunked(q[sl], k[sl], v[sl], w[h:h + 1], W.phi, W.eps, 256)
    assert W.rounds == 256
    total = np.zeros(W.B, dtype=np.int64)
    for rnd in range(W.rounds):
        qd, kd, vd = W.draft_inputs(rnd)
        parent, accept = W.trees(rnd)
        par, acc = torch.from_numpy(parent).cuda(), torch.from_numpy(accept).cuda()
        dq, dk, dv = dev(qd), dev(kd), dev(vd)
        before = st.clone() if rnd % 32 == 0 else None
        o = ctx.la_verify_tree(dq, dk, dv, par, dw, st)
        o0 = ctx.la_verify_tree(dq, dk, dv, par, dw0, st)
        if before is not None:
            assert torch.equal(st.S, before.S) and torch.equal(st.z, before.z) and torch.equal(st.win, before.win)
        path, clen = ctx.la_commit(dk, dv, par, acc, st)
        # integer outputs of every sequence against a parent walk done here
        hp, hl = path.cpu().numpy(), clen.cpu().numpy()
        for b in range(W.B):
            chain, m = [], int(accept[b])
            while m >= 0:
                chain.append(m)
                m = int(parent[b, m])
            chain.reverse()
            assert int(hl[b]) == len(chain)
            assert hp[b].tolist() == chain + [-1] * (W.max_depth - len(chain))
            total[b] += len(chain)
        for b, h in units:
            sl = (slice(b, b + 1), slice(h, h + 1))
            want = orc.verify_tree(qd[sl], kd[sl], vd[sl], parent[b:b + 1], w[h:h + 1], W.phi, W.eps, ost[(b, h)])
            assert rel_err(host(o[sl]), want) < TOL["bf16"], (rnd, b, h)
            la = orc.verify_tree(qd[sl], kd[sl], vd[sl], parent[b:b + 1], w0[h:h + 1], W.phi, W.eps, ost[(b, h)])
            assert rel_err(host(o0[sl]), la) < TOL["bf16"], (rnd, b, h)
            ost[(b, h)], _, _ = orc.commit(kd[sl], vd[sl], parent[b:b + 1], accept[b:b + 1], W.phi, ost[(b, h)],
                                           W.max_depth)
    for b, h in units:
        sl = (slice(b, b + 1), slice(h, h + 1))
        assert rel_err(host(st.S[sl]), ost[(b, h)].S) < TOL["bf16"]
        assert rel_err(host(st.z[sl]), ost[(b, h)].z) < TOL["bf16"]
        np.testing.assert_array_equal(host(st.win[sl]), ost[(b, h)].win)
        assert int(st.pos[b]) == int(ost[(b, h)].pos[0])
    assert st.pos.cpu().numpy().tolist() == (W.T + total).tolist()
    assert ctx.la_last_device_status() == binding.LA_OK


def test_tree_verify_taps8_full_size_rounds():
    """The 8-tap verify of the bench line at full size (512 units: more than four taps, summed beside the tensor
    cores): 12 rounds of verify + commit with the state carried, sampled units against the oracle, the window of 7
    rows bit-exact at the end."""
    W = wl.tree_verify_taps8()
    q, k, v = W.prefill_inputs()
    w = W.weights()
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, W.io, max_nodes=W.tree_nodes, max_depth=W.max_depth)
    st = ctx.new_state(W.B)
    dw = dev(w, "f32")
    ctx.la_prefill(dev(q), dev(k), dev(v), dw, st)
    units = ((0, 0), (5, 9), (9, 30), (15, 31))            # (15, 31): the last unit of the launch's last round
    ost = {}
    for b, h in units:
        sl = (slice(b, b + 1), slice(h, h + 1))
        _, ost[(b, h)] = orc.prefill_chunked(q[sl], k[sl], v[sl], w[h:h + 1], W.phi, W.eps, 256)
    for rnd in range(12):
        qd, kd, vd = W.draft_inputs(rnd)
        parent, accept = W.trees(rnd)
        par, acc = torch.from_numpy(parent).cuda(), torch.from_numpy(accept).cuda()
        dq, dk, dv = dev(qd), dev(kd), dev(vd)
        o = ctx.la_verify_tree(dq, dk, dv, par, dw, st)
        ctx.la_commit(dk, dv, par, acc, st)
        for b, h in units:
            sl = (slice(b, b + 1), slice(h, h + 1))
            want = orc.verify_tree(qd[sl], kd[sl], vd[sl], parent[b:b + 1], w[h:h + 1], W.phi, W.eps, ost[(b, h)])
            assert rel_err(host(o[sl]), want) < TOL["bf16"], (rnd, b, h)
            ost[(b, h)], _, _ = orc.commit(kd[sl], vd[sl], parent[b:b + 1], accept[b:b + 1], W.phi, ost[(b, h)],
                                           W.max_depth)
    for b, h in units:
        sl = (slice(b, b + 1), slice(h, h + 1))
        assert rel_err(host(st.S[sl]), ost[(b, h)].S) < TOL["bf16"]
        np.testing.assert_array_equal(host(st.win[sl]), ost[(b, h)].win)
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
