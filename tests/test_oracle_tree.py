"""Pins for the integer parts of the oracle: ancestor mask, greedy acceptance, KV commit.

Each check compares the oracle with something that is not the oracle: a hand-worked example
(tests/golden), a closed form (chain, star), a different algorithm (recurrence, numpy fancy
indexing) or brute force over every tree of at most 8 nodes."""
import itertools
import json
import os

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold(name):
    with open(os.path.join(GOLD, name)) as f:
        return json.load(f)


def all_parent_arrays(N):
    """Every valid parent array with N nodes: parent[i] in [0, i) for i >= 1 -> (N-1)! arrays."""
    for tail in itertools.product(*[range(i) for i in range(1, N)]):
        yield np.array((-1,) + tail, dtype=np.int32)


# ------------------------------------------------------------------ mask

def test_mask_hand_example():
    g = _gold("tree7.json")
    mask, depth, ok = oracle.tree_mask(np.array([g["parents"]], dtype=np.int32))
    assert ok
    assert [int(x) for x in mask[0, :, 0]] == [int(h, 16) for h in g["mask_hex"]]
    assert depth[0].tolist() == g["depth"]


@pytest.mark.parametrize("N", [1, 2, 31, 60, 64, 65, 128])
def test_mask_chain_is_lower_triangular(N):
    parents = np.arange(-1, N - 1, dtype=np.int32)[None]
    mask, depth, ok = oracle.tree_mask(parents)
    assert ok
    for i in range(N):
        full = (1 << (i + 1)) - 1
        got = sum(int(mask[0, i, w]) << (64 * w) for w in range(mask.shape[2]))
        assert got == full
    assert depth[0].tolist() == list(range(N))


@pytest.mark.parametrize("N", [2, 60, 100])
def test_mask_star(N):
    parents = np.zeros((1, N), dtype=np.int32)
    parents[0, 0] = -1
    mask, depth, ok = oracle.tree_mask(parents)
    assert ok
    for i in range(N):
        got = sum(int(mask[0, i, w]) << (64 * w) for w in range(mask.shape[2]))
        assert got == (1 | (1 << i))
    assert depth[0].tolist() == [0] + [1] * (N - 1)


def test_mask_exhaustive_up_to_8_nodes_matches_recurrence():
    for N in range(1, 9):
        arrays = np.stack(list(all_parent_arrays(N)))
        mask, depth, ok = oracle.tree_mask(arrays)
        assert ok
        for b in range(arrays.shape[0]):
            m = [0] * N
            d = [0] * N
            m[0] = 1
            for i in range(1, N):
                p = int(arrays[b, i])
                m[i] = m[p] | (1 << i)
                d[i] = d[p] + 1
            assert [int(x) for x in mask[b, :, 0]] == m
            assert depth[b].tolist() == d
            assert [bin(x).count("1") - 1 for x in m] == d


def test_mask_rejects_bad_parents_without_crashing():
    parents = np.array([[-1, 0, 5, 1], [-1, 0, 1, 2]], dtype=np.int32)
    mask, depth, ok = oracle.tree_mask(parents)
    assert not ok
    assert int(mask[0, 2, 0]) == 1 << 2          # offending row: self bit only
    assert int(mask[1, 3, 0]) == 0b1111          # the valid sequence is unaffected


# ------------------------------------------------------------------ acceptance

def test_accept_hand_example():
    g = _gold("tree7.json")
    path, alen, bonus = oracle.accept([g["draft_ids"]], [g["target_ids"]], [g["parents"]])
    assert alen[0] == g["accept_len"] and bonus[0] == g["bonus"]
    assert path[0, :alen[0]].tolist() == g["path"]
    assert (path[0, alen[0]:] == -1).all()
    matched = [i for i in range(1, 7) if g["draft_ids"][i] == g["target_ids"][g["parents"][i]]]
    assert matched == g["matched_nodes"]


def test_accept_duplicate_siblings_takes_the_longer_branch():
    g = _gold("dup_sibling.json")
    path, alen, bonus = oracle.accept([g["draft_ids"]], [g["target_ids"]], [g["parents"]])
    assert path[0, :alen[0]].tolist() == g["path"]
    assert alen[0] == g["accept_len"] and bonus[0] == g["bonus"]


def test_accept_nothing_matches_returns_root_only():
    parents = np.array([[-1, 0, 0, 1]], dtype=np.int32)
    path, alen, bonus = oracle.accept([[9, 1, 2, 3]], [[50, 51, 52, 53]], parents)
    assert alen[0] == 1 and path[0].tolist() == [0, -1, -1, -1] and bonus[0] == 50


def test_accept_root_draft_token_is_ignored():
    parents = np.array([[-1, 0, 1]], dtype=np.int32)
    a = oracle.accept([[111, 7, 8]], [[7, 8, 9]], parents)
    b = oracle.accept([[-5, 7, 8]], [[7, 8, 9]], parents)
    assert a[0].tolist() == b[0].tolist() == [[0, 1, 2]]
    assert a[1][0] == 3 and a[2][0] == 9


def _brute_force_accept(parents, matched):
    """Enumerate every root-to-node path explicitly and keep the best fully matched one."""
    N = len(parents)
    children = {i: [] for i in range(N)}
    for i in range(1, N):
        children[int(parents[i])].append(i)
    paths = []
    stack = [[0]]
    while stack:
        p = stack.pop()
        paths.append(p)
        for c in children[p[-1]]:
            stack.append(p + [c])
    best = None
    for p in paths:
        if all(matched[a] for a in p[1:]):
            key = (-len(p), p[-1])
            if best is None or key < best[0]:
                best = (key, p)
    return best[1]


def test_accept_exhaustive_up_to_8_nodes_matches_path_enumeration():
    for N in range(1, 9):
        arrays = list(all_parent_arrays(N))
        patterns = list(itertools.product([0, 1], repeat=N - 1))
        par_rows, dr_rows, tg_rows, want = [], [], [], []
        for parents in arrays:
            target = np.arange(100, 100 + N, dtype=np.int32)
            for pat in patterns:
                matched = (1,) + pat
                draft = np.full(N, 7, dtype=np.int32)
                for i in range(1, N):
                    if matched[i]:
                        draft[i] = target[parents[i]]
                par_rows.append(parents); dr_rows.append(draft); tg_rows.append(target)
                want.append(_brute_force_accept(parents, matched))
        path, alen, bonus = oracle.accept(np.stack(dr_rows), np.stack(tg_rows), np.stack(par_rows))
        for b, p in enumerate(want):
            assert alen[b] == len(p)
            assert path[b, :len(p)].tolist() == p
            assert (path[b, len(p):] == -1).all()
            assert bonus[b] == 100 + p[-1]


def test_accept_len_statistic_is_plausible():
    """tau = accept_len - 1 counts drafted tokens only (Sec. 5.1, 'average acceptance length');
    on the 60-node synthetic trees with p = 0.7 it should land in the paper's 2-3 range order."""
    from paper_2509_15235_b200 import synth
    rng = np.random.Generator(np.random.Philox(12345))
    taus = []
    for _ in range(200):
        parents = synth.draw_tree(60, 6, 4, rng)
        draft, target = synth.draw_ids(parents, 32000, 0.7, rng)
        _, alen, _ = oracle.accept(draft[None], target[None], parents[None])
        taus.append(int(alen[0]) - 1)
    assert 1.0 < np.mean(taus) < 5.0


# ------------------------------------------------------------------ compaction

def _random_cache(rng, B, Hkv, S_max, D):
    return rng.integers(0, 65536, size=(B, Hkv, S_max, D), dtype=np.int64).astype(np.uint16)


@pytest.mark.parametrize("path_list", [[0, 1, 2, 3], [0, 2, 3], [0, 1, 3, 6], [0, 7], [0], [0, 1, 2, 3, 4, 5, 6, 7],
                                        [0, 3, 5, 6, 7]])
def test_compact_matches_numpy_gather_then_scatter(path_list):
    rng = np.random.default_rng(5)
    B, Hkv, S_max, D, N, S = 2, 3, 40, 16, 8, 17
    k = _random_cache(rng, B, Hkv, S_max, D); v = _random_cache(rng, B, Hkv, S_max, D)
    L = len(path_list)
    path = np.full((B, N), -1, dtype=np.int32)
    path[:, :L] = path_list
    alen = np.full(B, L, dtype=np.int32)
    kv_len = np.array([S, S + 5], dtype=np.int32)
    k2, v2, len2 = oracle.kv_compact(k, v, path, alen, kv_len)
    for src, got in ((k, k2), (v, v2)):
        want = src.copy()
        for b in range(B):
            s = int(kv_len[b])
            want[b, :, s:s + L, :] = src[b][:, s + np.array(path_list), :]   # numpy gathers the RHS first
        assert np.array_equal(got, want)
    assert len2.tolist() == [S + L, S + 5 + L]


def test_compact_identity_path_changes_nothing_and_canaries_survive():
    rng = np.random.default_rng(6)
    k = _random_cache(rng, 1, 2, 64, 8); v = _random_cache(rng, 1, 2, 64, 8)
    path = np.full((1, 8), -1, dtype=np.int32); path[0, :4] = [0, 1, 2, 3]
    k2, v2, _ = oracle.kv_compact(k, v, path, [4], [30])
    assert np.array_equal(k, k2) and np.array_equal(v, v2)
    path[0, :3] = [0, 4, 7]; path[0, 3] = -1
    k3, v3, _ = oracle.kv_compact(k, v, path, [3], [30])
    assert np.array_equal(k3[:, :, :30], k[:, :, :30])          # prefix incl. canary row S-1
    assert np.array_equal(k3[:, :, 33:], k[:, :, 33:])          # everything past the accepted rows
    assert np.array_equal(k3[0, :, 31], k[0, :, 34]) and np.array_equal(v3[0, :, 32], v[0, :, 37])


def test_compact_overlap_hazard_is_gather_then_scatter():
    """path [0,2,3]: destination slot S+2 (k=2) is the source of k=1.  A sequential in-place copy
    in increasing k is still right here, one in decreasing k is not; the definition is order free."""
    k = np.arange(1 * 1 * 8 * 2, dtype=np.uint16).reshape(1, 1, 8, 2)
    path = np.array([[0, 2, 3, -1]], dtype=np.int32)
    k2, _, _ = oracle.kv_compact(k, k.copy(), path, [3], [2])
    assert k2[0, 0, 2:5].tolist() == [k[0, 0, 2].tolist(), k[0, 0, 4].tolist(), k[0, 0, 5].tolist()]
