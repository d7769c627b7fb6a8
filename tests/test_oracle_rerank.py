"""Pins of the tree-rerank oracle (CPU only): a hand-worked example, numpy's lexicographic sort, brute force over
every K-subset on small inputs, and the structural facts that cumulative log-probabilities guarantee (a kept
node's parent is kept; the output is a valid tree in parent-before-child order of the paper's size: 30 draft
tokens from a depth-3, width-8 expansion, App. A)."""
import itertools
import json
import os

import numpy as np

import oracle
from paper_2509_15235_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "rerank9.json")


def test_hand_worked_example():
    g = json.load(open(GOLDEN))
    parents, ids, sel, bad = oracle.tree_rerank([g["cand_parent"]], [g["cand_token"]], [g["cand_score"]], g["K"])
    assert bad == 0 and list(sel[0]) == g["selected"] and list(parents[0]) == g["parents"] and list(ids[0]) == g["draft_ids"]


def test_selection_is_numpys_sort_by_score_then_index():
    rng = np.random.Generator(np.random.Philox(1))
    B, M, K = 16, 200, 37
    score = np.round(rng.standard_normal((B, M)), 1).astype(np.float32)          # many exact ties
    parent = np.full((B, M), -1, dtype=np.int32)                                 # flat: every subset is closed
    token = rng.integers(0, 1000, size=(B, M)).astype(np.int32)
    parents, ids, sel, bad = oracle.tree_rerank(parent, token, score, K)
    assert bad == 0
    for b in range(B):
        order = np.lexsort((np.arange(M), -score[b].astype(np.float64)))
        want = np.sort(order[:K])
        assert np.array_equal(sel[b], want) and np.array_equal(ids[b, 1:], token[b, want])
        assert parents[b, 0] == -1 and np.all(parents[b, 1:] == 0)


def test_kept_set_has_the_largest_total_score_of_all_subsets():
    rng = np.random.Generator(np.random.Philox(2))
    M, K = 9, 4
    parent = np.full((1, M), -1, dtype=np.int32)
    for trial in range(30):
        score = rng.standard_normal((1, M)).astype(np.float32)
        _, _, sel, _ = oracle.tree_rerank(parent, np.zeros((1, M), np.int32), score, K)
        best = max(itertools.combinations(range(M), K), key=lambda c: float(score[0, list(c)].astype(np.float64).sum()))
        assert tuple(sel[0]) == best


def test_paper_sized_expansion_gives_a_valid_closed_tree():
    c = synth.make_rerank_candidates(B=6, depth=3, width=8, vocab=32000, seed=3)
    assert c["cand_parent"].shape == (6, 136)
    K = 30
    parents, ids, sel, bad = oracle.tree_rerank(c["cand_parent"], c["cand_token"], c["cand_score"], K)
    assert bad == 0
    mask, depth, ok = oracle.tree_mask(parents)
    assert ok and depth.max() <= 3 and np.all(np.diff(sel, axis=1) > 0)
    for b in range(6):
        kept = set(sel[b].tolist())
        for j in range(1, K + 1):
            cp = c["cand_parent"][b, sel[b, j - 1]]
            assert (cp == -1 and parents[b, j] == 0) or (cp in kept and sel[b, parents[b, j] - 1] == cp)
            assert ids[b, j] == c["cand_token"][b, sel[b, j - 1]]
        # nothing left out scores higher than something kept
        out = [i for i in range(136) if i not in kept]
        assert c["cand_score"][b, out].max() <= c["cand_score"][b, sel[b]].min()


def test_nan_scores_rank_last_and_broken_inputs_are_flagged():
    score = np.array([[np.nan, -1.0, -2.0, np.nan, -0.5]], dtype=np.float32)
    parent = np.full((1, 5), -1, dtype=np.int32)
    _, _, sel, bad = oracle.tree_rerank(parent, np.zeros((1, 5), np.int32), score, 3)
    assert bad == 0 and list(sel[0]) == [1, 2, 4]
    _, _, sel, _ = oracle.tree_rerank(parent, np.zeros((1, 5), np.int32), score, 4)
    assert list(sel[0]) == [0, 1, 2, 4]
    # a child that outscores its parent, so that the parent is dropped: flagged, parents all -1
    parents, ids, sel, bad = oracle.tree_rerank([[-1, 0, -1]], [[5, 6, 7]], np.array([[-3.0, -1.0, -2.0]], np.float32), 2)
    assert bad == 1 and list(sel[0]) == [1, 2] and list(parents[0]) == [-1, -1, -1] and list(ids[0]) == [0, 6, 7]
    # a parent index that is not an earlier candidate
    parents, _, _, bad = oracle.tree_rerank([[-1, 1, 0]], [[5, 6, 7]], np.array([[-1.0, -2.0, -3.0]], np.float32), 3)
    assert bad == 1 and list(parents[0]) == [-1, -1, -1, -1]
    # K = M keeps everything, K = 0 keeps the root only
    parents, ids, sel, bad = oracle.tree_rerank([[-1, 0, 1]], [[5, 6, 7]], np.array([[-1.0, -2.0, -3.0]], np.float32), 3)
    assert bad == 0 and list(parents[0]) == [-1, 0, 1, 2]
    parents, ids, sel, bad = oracle.tree_rerank([[-1, 0, 1]], [[5, 6, 7]], np.array([[-1.0, -2.0, -3.0]], np.float32), 0)
    assert bad == 0 and parents.shape == (1, 1) and parents[0, 0] == -1
