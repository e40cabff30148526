"""la_accept_threshold (Sec. 4.2: accept, reject, resample) against the oracle: bit-exact integers."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import la_oracle as orc
from paper_2406_07368_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu


def cu(x):
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def scores(seed, rnd, B, N, ties=False):
    g = wl.rng(seed, 7, rnd)
    score = g.uniform(0.0, 1.5, size=(B, N)).astype(np.float32)
    thresh = g.uniform(0.0, 1.0, size=(B, N)).astype(np.float32)
    if ties:                                   # a third of the nodes sit exactly on their threshold
        pick = g.uniform(size=(B, N)) < 0.33
        thresh[pick] = score[pick]
    return score, thresh


@pytest.mark.parametrize("B,N,depth", [(7, 64, 5), (1, 1, 1), (13, 37, 8), (4, 64, 64), (130, 20, 4)])
def test_accept_threshold_is_bit_exact(B, N, depth):
    ctx = binding.Context(2, 128, 3, "elu1", 0.0, "bf16", max_nodes=64, max_depth=64)
    for rnd in range(3):
        parent = np.stack([wl.chain_tree(N)] * B) if depth == 64 else wl.tree_batch(31 + N, rnd, B, N, max_depth=depth)[0]
        score, thresh = scores(31 + N, rnd, B, N, ties=rnd == 2)
        if depth == 64:
            score = score + 0.9                # long accepted chains
        want = orc.accept_threshold(parent, score, thresh)
        got = ctx.la_accept_threshold(cu(parent.astype(np.int32)), cu(score), cu(thresh))
        assert ctx.la_last_device_status() == binding.LA_OK
        for g, w_ in zip(got, want):
            np.testing.assert_array_equal(g.cpu().numpy(), w_)


def test_hand_worked_example_and_nan():
    g = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_example_accept_threshold.json")))
    ctx = binding.Context(2, 128, 3, "elu1", 0.0, "bf16", max_nodes=16)
    parent = cu(np.array([g["parent"]], dtype=np.int32))
    node, length = ctx.la_accept_threshold(parent, cu(np.array([g["score"]], dtype=np.float32)),
                                           cu(np.array([g["thresh"]], dtype=np.float32)))
    assert (int(node[0]), int(length[0])) == (g["accept_node"], g["accept_len"])
    score = np.array([g["score"]], dtype=np.float32)
    score[0, 3] = np.nan                       # node 3 can no longer pass: its subtree is out
    want = orc.accept_threshold(np.array([g["parent"]]), score, np.array([g["thresh"]], dtype=np.float32))
    node, length = ctx.la_accept_threshold(parent, cu(score), cu(np.array([g["thresh"]], dtype=np.float32)))
    assert (int(node[0]), int(length[0])) == (int(want[0][0]), int(want[1][0])) == (2, 2)


def test_accept_threshold_with_a_zero_one_score_is_the_greedy_rule_and_feeds_commit():
    B, N = 6, 40
    parent, _ = wl.tree_batch(41, 0, B, N, max_depth=6)
    draft, pred_root, pred = wl.token_batch(41, 0, B, N, vocab=2)
    above = np.where(parent < 0, pred_root[:, None], np.take_along_axis(pred, np.maximum(parent, 0), axis=1))
    score = (draft == above).astype(np.float32)
    ctx = binding.Context(2, 128, 3, "elu1", 0.0, "bf16", max_nodes=64, max_depth=8)
    par = cu(parent.astype(np.int32))
    node, length = ctx.la_accept_threshold(par, cu(score), cu(np.full((B, N), 0.5, dtype=np.float32)))
    gnode, glen, _ = ctx.la_accept_greedy(par, cu(draft), cu(pred_root), cu(pred))
    assert torch.equal(node, gnode) and torch.equal(length, glen)


def test_accept_threshold_flags_bad_trees_and_rejects_bad_arguments():
    B, N = 3, 8
    parent, _ = wl.tree_batch(5, 0, B, N)
    score, thresh = np.ones((B, N), dtype=np.float32), np.zeros((B, N), dtype=np.float32)
    bad = parent.copy()
    bad[1, 2] = 6                                                          # parent after child
    ctx = binding.Context(2, 128, 3, "elu1", 0.0, "bf16", max_nodes=8)
    node, length = ctx.la_accept_threshold(cu(bad.astype(np.int32)), cu(score), cu(thresh))
    assert ctx.la_last_device_status() == binding.LA_ERR_BAD_TREE
    assert int(node[1]) == -1 and int(length[1]) == 0
    want = orc.accept_threshold(parent[[0, 2]], score[[0, 2]], thresh[[0, 2]])
    np.testing.assert_array_equal(node[[0, 2]].cpu().numpy(), want[0])
    np.testing.assert_array_equal(length[[0, 2]].cpu().numpy(), want[1])
    ctx.la_clear_device_status()
    n0 = ctx.la_launch_count()
    with pytest.raises(binding.LaError) as e:                               # more nodes than the context allows
        ctx.la_accept_threshold(torch.zeros(1, 9, dtype=torch.int32, device="cuda"),
                                torch.zeros(1, 9, device="cuda"), torch.zeros(1, 9, device="cuda"))
    assert e.value.code == binding.LA_ERR_INVALID_ARG and ctx.la_launch_count() == n0
