"""The seeded input generators: reproducible, order-independent, valid trees, exact bf16 rounding."""
import numpy as np
import torch

from paper_2406_07368_b200 import workloads as wl


def test_bf16_rounding_matches_torch():
    x = np.random.default_rng(0).standard_normal(100000).astype(np.float32) * 3
    x[:4] = [0.0, -0.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8]     # ties
    want = torch.from_numpy(x).to(torch.bfloat16).float().numpy()
    np.testing.assert_array_equal(wl.round_to_bf16(x), want)


def test_draws_do_not_depend_on_call_order():
    w = wl.tree_verify()
    a = w.draft_inputs(3, B=2, H=2)
    _ = w.draft_inputs(1, B=2, H=2)
    b = w.draft_inputs(3, B=2, H=2)
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x, y)
    assert not np.array_equal(a[0], a[1])
    p1, a1 = w.trees(5, B=3)
    p2, a2 = w.trees(5, B=3)
    np.testing.assert_array_equal(p1, p2)
    np.testing.assert_array_equal(a1, a2)


def test_trees_are_valid():
    w = wl.tree_verify()
    for r in range(4):
        parent, accept = w.trees(r, B=4)
        assert parent.shape == (4, 64) and parent.dtype == np.int32
        for b in range(4):
            depth = wl.tree_depths(parent[b])
            assert all(-1 <= parent[b, n] < n for n in range(64))
            assert depth.max() <= 5
            fan = np.bincount(parent[b][parent[b] >= 0], minlength=64)
            assert fan.max() <= 4 and (parent[b] < 0).sum() <= 4
            assert 0 <= accept[b] < 64 and 1 <= depth[accept[b]] <= 5


def test_workload_shapes():
    w = wl.llama7b_prefill()
    q, k, v = w.prefill_inputs(B=1, H=2, T=16)
    assert q.shape == (1, 2, 16, 128) and q.dtype == np.float32
    np.testing.assert_array_equal(q, wl.round_to_bf16(q))
    assert abs(float(q.std()) - 128 ** -0.5) < 0.01
    cw = w.weights()
    assert cw.shape == (32, 128, 3) and abs(float(cw.var()) - 1 / 3) < 0.02
    assert set(wl.WORKLOADS) == {"tiny_fp32", "llama7b_prefill", "batched_decode", "tree_verify", "long_prefill",
                                 "prompt_gen", "grouped_block", "prefill_taps32", "tree_verify_taps8"}
