"""Pins of oracle.accept_threshold (Sec. 4.2: accept, reject, resample) against things other than itself: a
hand-worked example, the greedy rule it contains as a special case, the closed form of rejection sampling along a
chain, brute force over all root paths, and planted mistakes."""
import json
import os

import numpy as np
import pytest

from oracle import la_oracle as orc
from paper_2406_07368_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_example_accept_threshold.json")


def f32(x):
    return np.asarray(x, dtype=np.float32)


def test_hand_worked_example():
    g = json.load(open(GOLDEN))
    parent = np.array([g["parent"]])
    node, length = orc.accept_threshold(parent, f32([g["score"]]), f32([g["thresh"]]))
    assert (int(node[0]), int(length[0])) == (g["accept_node"], g["accept_len"])
    th = list(g["thresh"])
    th[5] = g["thresh5_second"]
    node, length = orc.accept_threshold(parent, f32([g["score"]]), f32([th]))
    assert (int(node[0]), int(length[0])) == (g["accept_node_second"], g["accept_len_second"])
    th = list(g["thresh"])
    th[0] = g["thresh0_third"]
    node, length = orc.accept_threshold(parent, f32([g["score"]]), f32([th]))
    assert (int(node[0]), int(length[0])) == (g["accept_node_third"], g["accept_len_third"])


@pytest.mark.parametrize("seed", range(6))
def test_greedy_rule_is_the_special_case_of_a_zero_one_score(seed):
    """score = 1 where the drafted token is the verifier's token at the node above, else 0; threshold 1/2: the same
    nodes as accept_greedy (which is pinned by its own golden file and path enumeration)."""
    B, N = 5, 1 + 9 * seed
    parent, _ = wl.tree_batch(50 + seed, 0, B, N, max_depth=6)
    draft, pred_root, pred = wl.token_batch(60 + seed, 0, B, N, vocab=3)
    above = np.where(parent < 0, np.asarray(pred_root)[:, None], np.take_along_axis(np.asarray(pred), np.maximum(parent, 0), axis=1))
    score = f32(np.asarray(draft) == above)
    want_node, want_len, _ = orc.accept_greedy(parent, draft, pred_root, pred)
    node, length = orc.accept_threshold(parent, score, np.full((B, N), 0.5, dtype=np.float32))
    np.testing.assert_array_equal(node, want_node)
    np.testing.assert_array_equal(length, want_len)


@pytest.mark.parametrize("N", [1, 2, 7, 64])
def test_rejection_sampling_along_a_chain_stops_at_the_first_failed_draw(N):
    """A chain is the original speculative sampling: the accepted length is the index of the first token whose uniform
    draw exceeds p/q (all of them if none does)."""
    g = wl.rng(70, 1, N)
    B = 9
    ratio = f32(g.uniform(0.0, 1.6, size=(B, N)))
    u = f32(g.uniform(0.0, 1.0, size=(B, N)))
    parent = np.tile(wl.chain_tree(N), (B, 1))
    node, length = orc.accept_threshold(parent, ratio, u)
    for b in range(B):
        fails = np.nonzero(~(ratio[b] >= u[b]))[0]
        first = int(fails[0]) if len(fails) else N
        assert int(length[b]) == first and int(node[b]) == first - 1


@pytest.mark.parametrize("seed", range(5))
def test_brute_force_over_all_root_paths(seed):
    N = 12
    parent, _ = wl.tree_batch(80 + seed, 0, 3, N, max_depth=5)
    g = wl.rng(81, 2, seed)
    score = f32(g.uniform(size=(3, N)))
    thresh = f32(g.uniform(0.0, 0.6, size=(3, N)))
    node, length = orc.accept_threshold(parent, score, thresh)
    for b in range(3):
        best, best_len = -1, 0
        for n in range(N):
            path, m = [], n
            while m >= 0:
                path.append(m)
                m = int(parent[b, m])
            if all(score[b, m] >= thresh[b, m] for m in path) and len(path) > best_len:
                best, best_len = n, len(path)
        assert (int(node[b]), int(length[b])) == (best, best_len)


def test_nan_never_passes_and_bad_trees_are_refused():
    parent = np.array([[-1, 0, 1]])
    node, length = orc.accept_threshold(parent, f32([[1.0, np.nan, 1.0]]), f32([[0.0, 0.0, 0.0]]))
    assert (int(node[0]), int(length[0])) == (0, 1)
    node, length = orc.accept_threshold(parent, f32([[1.0, 1.0, 1.0]]), f32([[0.0, np.nan, 0.0]]))
    assert (int(node[0]), int(length[0])) == (0, 1)
    with pytest.raises(ValueError):
        orc.accept_threshold(np.array([[-1, 1, 0]]), f32([[1, 1, 1]]), f32([[0, 0, 0]]))


def test_planted_mistakes_are_caught():
    """A strict comparison, a missing parent condition and a largest-index tie-break each fail the hand example."""
    g = json.load(open(GOLDEN))
    parent, score, thresh = np.array(g["parent"]), f32(g["score"]), f32(g["thresh"])

    def variant(strict=False, ignore_parent=False, last_wins=False, th=thresh):
        acc, depth, best, bd = {}, {}, -1, 0
        for n, p in enumerate(parent):
            ok = score[n] > th[n] if strict else score[n] >= th[n]
            acc[n] = ok and (ignore_parent or p < 0 or acc[p])
            depth[n] = 1 if p < 0 else depth[p] + 1
            if acc[n] and (depth[n] >= bd if last_wins else depth[n] > bd) and depth[n] > 0:
                best, bd = n, depth[n]
        return best, bd
    assert variant() == (g["accept_node"], g["accept_len"])
    assert variant(strict=True) != (g["accept_node"], g["accept_len"])            # node 3 sits exactly on its threshold
    assert variant(ignore_parent=True) != (g["accept_node"], g["accept_len"])     # node 8 passes on its own, at depth 4
    assert variant(last_wins=True) != (g["accept_node"], g["accept_len"])         # nodes 6 and 9 tie at depth 3
    th2 = thresh.copy()
    th2[5] = g["thresh5_second"]
    assert variant(th=th2) == (g["accept_node_second"], g["accept_len_second"])
