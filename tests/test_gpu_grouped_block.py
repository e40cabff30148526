"""Parity of la_prefill_grouped (the three-branch block of Sec. 4.1) with the float64 oracle, element by element."""
import numpy as np
import pytest
import torch

from oracle import la_oracle as orc
from paper_2406_07368_b200 import binding, workloads as wl
from tests._util import TOL, rel_err, rel_err_group_octaves

pytestmark = pytest.mark.gpu


def dev(x, io):
    return torch.from_numpy(np.ascontiguousarray(x)).to(binding.TORCH_DTYPE[io]).cuda()


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64) if t.is_floating_point() else t.cpu().numpy()


def check_state(st, wst, io):
    assert rel_err(host(st.S), wst.S) < TOL[io] and rel_err(host(st.z), wst.z) < TOL[io]
    np.testing.assert_array_equal(host(st.win), wst.win)
    np.testing.assert_array_equal(host(st.pos), wst.pos)


@pytest.mark.parametrize("io,d,phi,eps,W,T,C,alpha,v_mean,zero_w", [
    ("bf16", 128, "elu1", 0.0, 3, 700, 64, 1.0, 0.0, False),      # the paper's group size for LLaMA
    ("bf16", 128, "elu1", 0.0, 3, 700, 128, 0.5, 1.0, False),
    ("bf16", 128, "relu", 1e-6, 5, 333, 100, 0.7, 0.0, True),     # a group size that is no multiple of the query block
    ("bf16", 64, "elu1", 0.0, 3, 600, 256, 1.0, 1.0, True),       # FLASH's group size
    ("f32", 64, "elu1", 0.0, 3, 256, 64, 1.0, 0.0, False),
    ("f32", 128, "relu", 1e-6, 4, 150, 64, 0.3, 1.0, False),
    ("f32", 64, "elu1", 0.0, 32, 200, 37, 1.0, 0.0, False),       # the longest tap window, reaching across groups
    ("bf16", 128, "elu1", 0.0, 1, 50, 1, 1.0, 1.0, False),        # every token its own group
    ("bf16", 128, "elu1", 0.0, 3, 90, 128, 0.9, 0.0, False),      # one group holds the whole sequence
    ("bf16", 128, "elu1", 0.0, 3, 1, 64, 1.0, 0.0, False),
])
def test_grouped_block_matches_oracle(io, d, phi, eps, W, T, C, alpha, v_mean, zero_w):
    B, H = 2, 3
    scale_in = 1.0 if io == "f32" else 0.5
    q, k, v = wl.qkv(3000 + T + C, (B, H, T, d), scale_in, io, v_mean=v_mean)
    w = wl.conv_weights(T + C, H, d, W)
    if zero_w:
        w = np.zeros_like(w)
    ctx = binding.Context(H, d, W, phi, eps, io)
    assert C <= ctx.la_prefill_grouped_max_group()
    st = ctx.new_state(B)
    st.S.fill_(5.0)                                   # a fresh call ignores what the buffers hold
    o = ctx.la_prefill_grouped(dev(q, io), dev(k, io), dev(v, io), dev(w, "f32"), st, C, alpha, d ** -0.5)
    assert ctx.la_last_device_status() == binding.LA_OK
    want, wst = orc.prefill_grouped_block(q, k, v, w, phi, eps, C, alpha, d ** -0.5)
    if zero_w and v_mean == 0.0 and io == "bf16":     # zero taps, zero-mean values: one scale per octave of the group
        assert rel_err_group_octaves(host(o), want, C) < TOL[io]
    else:
        assert rel_err(host(o), want) < TOL[io]
    if T > 2 * C and not (zero_w and v_mean == 0.0):  # beyond the first group the global branch is at work
        assert rel_err(host(o)[:, :, C:], want[:, :, C:]) < TOL[io]
    check_state(st, wst, io)


@pytest.mark.parametrize("io,C,cut_groups,T", [("bf16", 64, 3, 500), ("f32", 32, 2, 131)])
def test_grouped_block_continues_at_a_group_boundary(io, C, cut_groups, T):
    B, H, d, W, alpha = 1, 2, 128 if io == "bf16" else 64, 4, 0.8
    q, k, v = wl.qkv(3100 + T, (B, H, T, d), 0.5, io, v_mean=0.5)
    w = wl.conv_weights(T, H, d, W)
    ctx = binding.Context(H, d, W, "elu1", 0.0, io)
    st = ctx.new_state(B)
    cut = cut_groups * C
    sl = lambda x, a, b: dev(x[:, :, a:b], io)
    o1 = ctx.la_prefill_grouped(sl(q, 0, cut), sl(k, 0, cut), sl(v, 0, cut), dev(w, "f32"), st, C, alpha, 0.1)
    o2 = ctx.la_prefill_grouped(sl(q, cut, T), sl(k, cut, T), sl(v, cut, T), dev(w, "f32"), st, C, alpha, 0.1,
                                init_state=True)
    want, wst = orc.prefill_grouped_block(q, k, v, w, "elu1", 0.0, C, alpha, 0.1)
    assert rel_err(host(torch.cat([o1, o2], dim=2)), want) < TOL[io]
    assert rel_err(host(o2), want[:, :, cut:]) < TOL[io]
    check_state(st, wst, io)
    # the state is the plain running state: a decode step of the exact layer can follow
    qs, ks, vs = wl.qkv(3200, (B, H, d), 0.5, io)
    od = ctx.la_decode_step(dev(qs, io), dev(ks, io), dev(vs, io), dev(w, "f32"), st)
    wd, _ = orc.decode_step(qs, ks, vs, w, "elu1", 0.0, wst)
    assert rel_err(host(od), wd) < TOL[io]


def test_grouped_block_alpha_zero_and_a_single_group_agree_with_library_softmax_attention():
    """Against torch's softmax attention on the GPU inputs (a library routine, not the oracle): alpha = 0 leaves
    softmax attention group by group plus the convolution; here the taps are zero as well."""
    io, B, H, d, T, C, W = "bf16", 1, 2, 128, 256, 64, 3
    q, k, v = wl.qkv(3300, (B, H, T, d), 0.5, io)
    w = np.zeros((H, d, W), dtype=np.float32)
    ctx = binding.Context(H, d, W, "elu1", 0.0, io)
    o = ctx.la_prefill_grouped(dev(q, io), dev(k, io), dev(v, io), dev(w, "f32"), ctx.new_state(B), C, 0.0, d ** -0.5)
    tq, tk, tv = (torch.from_numpy(x).double().view(B, H, T // C, C, d) for x in (q, k, v))
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=d ** -0.5)
    assert rel_err(host(o), want.reshape(B, H, T, d).numpy()) < TOL[io]


def test_grouped_block_full_head_count_more_chains_than_sms():
    """LLaMA-2-7B geometry with the paper's group size of 64: 160 chains on 148 SMs, sampled units against the oracle."""
    io, B, H, d, T, C, W = "bf16", 5, 32, 128, 1024, 64, 3
    q, k, v = wl.qkv(3400, (B, H, T, d), d ** -0.5, io)
    w = wl.conv_weights(3400, H, d, W)
    ctx = binding.Context(H, d, W, "elu1", 0.0, io)
    st = ctx.new_state(B)
    o = ctx.la_prefill_grouped(dev(q, io), dev(k, io), dev(v, io), dev(w, "f32"), st, C, 1.0, d ** -0.5)
    assert ctx.la_last_device_status() == binding.LA_OK
    for b, h in ((0, 0), (2, 17), (4, 19), (4, 31)):
        sl = (slice(b, b + 1), slice(h, h + 1))
        want, wst = orc.prefill_grouped_block(q[sl], k[sl], v[sl], w[h:h + 1], "elu1", 0.0, C, 1.0, d ** -0.5)
        assert rel_err(host(o[sl]), want) < TOL[io], (b, h)
        assert rel_err(host(st.S[sl]), wst.S) < TOL[io] and rel_err(host(st.z[sl]), wst.z) < TOL[io]
    assert st.pos.tolist() == [T] * B


def test_grouped_block_rejects_groups_beyond_what_the_kernel_holds():
    ctx = binding.Context(2, 128, 3, "elu1", 0.0, "bf16")
    assert ctx.la_prefill_grouped_max_group() == 128
    x = torch.zeros(1, 2, 300, 128, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(2, 128, 3, device="cuda")
    with pytest.raises(binding.LaError) as e:
        ctx.la_prefill_grouped(x, x, x, w, ctx.new_state(1), 256, 1.0, 0.1)
    assert e.value.code == binding.LA_ERR_UNSUPPORTED
    with pytest.raises(binding.LaError) as e:
        ctx.la_prefill_grouped(x, x, x, w, ctx.new_state(1), 0, 1.0, 0.1)
    assert e.value.code == binding.LA_ERR_INVALID_ARG
    assert ctx.la_launch_count() == 0


@pytest.mark.parametrize("W", [1, 8, 20])
@pytest.mark.parametrize("C", [128, 48])
def test_grouped_block_on_tensor_cores_with_other_tap_windows(C, W):
    """Every window but 3 taps takes the long epilogue in the three-branch mode of the tensor-core kernel; a second
    call continues from the state and the window of the first."""
    io, d, B, H, T, alpha = "bf16", 128, 2, 2, 3 * 128 + 50, 0.6
    q, k, v = wl.qkv(3300 + C + W, (B, H, T, d), 0.5, io, v_mean=0.5)
    w = wl.conv_weights(3300 + W, H, d, W)
    ctx = binding.Context(H, d, W, "elu1", 0.0, io)
    st = ctx.new_state(B)
    cut = 2 * C
    sl = lambda x, a, b: dev(x[:, :, a:b], io)
    o1 = ctx.la_prefill_grouped(sl(q, 0, cut), sl(k, 0, cut), sl(v, 0, cut), dev(w, "f32"), st, C, alpha, d ** -0.5)
    o2 = ctx.la_prefill_grouped(sl(q, cut, T), sl(k, cut, T), sl(v, cut, T), dev(w, "f32"), st, C, alpha, d ** -0.5,
                                init_state=True)
    assert ctx.la_last_device_status() == binding.LA_OK
    want, wst = orc.prefill_grouped_block(q, k, v, w, "elu1", 0.0, C, alpha, d ** -0.5)
    assert rel_err(host(torch.cat([o1, o2], dim=2)), want) < TOL[io]
    check_state(st, wst, io)


@pytest.mark.parametrize("kernel", [0, 1])
@pytest.mark.parametrize("phi,eps,W,T,alpha,v_mean,zero_w", [
    ("elu1", 0.0, 3, 700, 1.0, 0.0, False), ("elu1", 0.0, 3, 700, 0.5, 1.0, True), ("relu", 1e-6, 5, 333, 0.7, 1.0, False),
    ("elu1", 0.0, 3, 128, 1.0, 0.0, False), ("elu1", 0.0, 3, 129, 1.0, 1.0, False), ("elu1", 0.0, 3, 1, 1.0, 0.0, False),
    ("relu", 0.0, 1, 400, 2.0, 1.0, False), ("elu1", 0.0, 16, 300, 1.0, 0.0, False), ("elu1", 0.0, 3, 2048, 1.0, 1.0, True),
    ("elu1", 0.0, 3, 500, 0.0, 1.0, False)])
@pytest.mark.parametrize("C", [128, 64, 100, 32])
def test_grouped_block_with_groups_of_one_tile_on_both_kernels(C, kernel, phi, eps, W, T, alpha, v_mean, zero_w):
    """Groups of 32 to 128 tokens with bf16 and d = 128: the tensor-core kernel (0; a shorter group takes a partly
    filled tile) and the CUDA-core kernel (1)."""
    io, B, H, d = "bf16", 2, 3, 128
    q, k, v = wl.qkv(5000 + T + W, (B, H, T, d), 0.5, io, v_mean=v_mean)
    w = wl.conv_weights(T + W, H, d, W)
    if zero_w:
        w = np.zeros_like(w)
    ctx = binding.Context(H, d, W, phi, eps, io)
    ctx.la_set_prefill_kernel(kernel)
    st = ctx.new_state(B)
    o = ctx.la_prefill_grouped(dev(q, io), dev(k, io), dev(v, io), dev(w, "f32"), st, C, alpha, d ** -0.5)
    assert ctx.la_last_device_status() == binding.LA_OK
    want, wst = orc.prefill_grouped_block(q, k, v, w, phi, eps, C, alpha, d ** -0.5)
    assert rel_err(host(o), want) < TOL[io]
    if T > 2 * C:
        assert rel_err(host(o)[:, :, C:], want[:, :, C:]) < TOL[io]
        assert rel_err(host(o)[:, :, -C:], want[:, :, -C:]) < TOL[io]
    check_state(st, wst, io)


@pytest.mark.parametrize("kernel", [0, 1])
def test_grouped_block_of_one_tile_continues_and_hands_over_to_decode(kernel):
    io, B, H, d, C, W, T, cut = "bf16", 1, 2, 128, 128, 4, 900, 384
    q, k, v = wl.qkv(5100, (B, H, T, d), 0.5, io, v_mean=0.5)
    w = wl.conv_weights(5100, H, d, W)
    ctx = binding.Context(H, d, W, "elu1", 0.0, io)
    ctx.la_set_prefill_kernel(kernel)
    st = ctx.new_state(B)
    sl = lambda x, a, b: dev(x[:, :, a:b], io)
    o1 = ctx.la_prefill_grouped(sl(q, 0, cut), sl(k, 0, cut), sl(v, 0, cut), dev(w, "f32"), st, C, 0.8, 0.1)
    o2 = ctx.la_prefill_grouped(sl(q, cut, T), sl(k, cut, T), sl(v, cut, T), dev(w, "f32"), st, C, 0.8, 0.1, init_state=True)
    want, wst = orc.prefill_grouped_block(q, k, v, w, "elu1", 0.0, C, 0.8, 0.1)
    assert rel_err(host(torch.cat([o1, o2], dim=2)), want) < TOL[io]
    assert rel_err(host(o2), want[:, :, cut:]) < TOL[io]
    check_state(st, wst, io)
    qs, ks, vs = wl.qkv(5101, (B, H, d), 0.5, io)
    od = ctx.la_decode_step(dev(qs, io), dev(ks, io), dev(vs, io), dev(w, "f32"), st)
    wd, _ = orc.decode_step(qs, ks, vs, w, "elu1", 0.0, wst)
    assert rel_err(host(od), wd) < TOL[io]
