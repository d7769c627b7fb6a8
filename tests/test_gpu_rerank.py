"""GPU parity (bit-exact) of the tree rerank against the oracle, through the C ABI, and the chain
rerank -> mask build -> sampled acceptance on its output."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_15235_b200 import synth

pytestmark = pytest.mark.gpu


def _run(cand_parent, cand_token, cand_score, K, N_max=None):
    from paper_2509_15235_b200 import binding
    import gpu_util as gu
    B, M = cand_parent.shape
    ctx = binding.VerifyContext(max(B, 1), N_max or max(K + 1, 1), 4, 4, 64, 256, 1)
    parents = torch.full((B, K + 1), -9, dtype=torch.int32, device="cuda")
    ids = torch.full((B, K + 1), -9, dtype=torch.int32, device="cuda")
    sel = torch.full((B, K), -9, dtype=torch.int32, device="cuda") if K > 0 else None
    score = torch.from_numpy(np.ascontiguousarray(cand_score, dtype=np.float32)).cuda()
    ctx.tree_rerank(gu.i32_dev(cand_parent), gu.i32_dev(cand_token), score, K, parents, ids, sel)
    torch.cuda.synchronize()
    status = ctx.status_poll()
    ctx.close()
    return parents.cpu().numpy(), ids.cpu().numpy(), (sel.cpu().numpy() if K > 0 else np.zeros((B, 0), np.int32)), status


def _check(cp, ct, cs, K, want_bad=0):
    got = _run(np.asarray(cp, np.int32), np.asarray(ct, np.int32), np.asarray(cs, np.float32), K)
    want = oracle.tree_rerank(cp, ct, cs, K)
    assert want[3] == want_bad and got[3] == (0 if want_bad == 0 else -8)
    for g, w in zip(got[:3], want[:3]):
        assert np.array_equal(g, w)
    return want


@pytest.mark.parametrize("depth,width,K,B", [(3, 8, 30, 4), (3, 8, 59, 1), (6, 4, 59, 8), (2, 8, 8, 2), (5, 16, 127, 3)])
def test_rerank_matches_the_oracle_on_level_by_level_expansions(depth, width, K, B):
    c = synth.make_rerank_candidates(B, depth, width, 32000, 40 + depth * width)
    parents, ids, sel, _ = _check(c["cand_parent"], c["cand_token"], c["cand_score"], K)
    assert oracle.tree_mask(parents)[2]


def test_rerank_ties_nan_zero_signs_ragged_sizes():
    rng = np.random.Generator(np.random.Philox(8))
    for M, K in [(1, 1), (1, 0), (7, 3), (255, 100), (256, 127), (257, 64), (600, 127), (2048, 127)]:
        B = 5
        score = np.round(rng.standard_normal((B, M)), 1).astype(np.float32)      # many ties, +0.0 and -0.0 among them
        score[0, rng.integers(0, M, size=max(1, M // 7))] = np.nan
        score[1, :] = -1.0                                                        # all equal: lowest indices win
        score[2, ::2] *= 0.0
        parent = np.full((B, M), -1, dtype=np.int32)
        token = rng.integers(0, 50000, size=(B, M)).astype(np.int32)
        _check(parent, token, score, K)


def test_rerank_flags_broken_inputs():
    _check([[-1, 0, -1]], [[5, 6, 7]], [[-3.0, -1.0, -2.0]], 2, want_bad=1)     # child outscores its parent
    _check([[-1, 1, 0]], [[5, 6, 7]], [[-1.0, -2.0, -3.0]], 3, want_bad=1)      # parent is not an earlier candidate
    _check([[-1, 0, -2]], [[5, 6, 7]], [[-1.0, -2.0, -3.0]], 1, want_bad=1)


def test_rerank_feeds_mask_build_and_sampled_acceptance():
    """The paper's sizes end to end: 136 candidates -> 30 draft tokens -> mask and sampled acceptance, each
    stage equal to the oracle run on the oracle's own output of the stage before."""
    from paper_2509_15235_b200 import binding
    import gpu_util as gu
    B, K, V = 3, 30, 32000
    N = K + 1
    c = synth.make_rerank_candidates(B, 3, 8, V, 77)
    want_parents, want_ids, _, bad = oracle.tree_rerank(c["cand_parent"], c["cand_token"], c["cand_score"], K)
    assert bad == 0
    s = synth.make_sampled_inputs(want_parents, V, 78)
    ctx = binding.VerifyContext(B, N, 4, 4, 64, 256, 1)
    parents = torch.zeros((B, N), dtype=torch.int32, device="cuda")
    ids = torch.zeros((B, N), dtype=torch.int32, device="cuda")
    sel = torch.zeros((B, K), dtype=torch.int32, device="cuda")
    f32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    ctx.tree_rerank(gu.i32_dev(c["cand_parent"]), gu.i32_dev(c["cand_token"]), f32(c["cand_score"]), K, parents, ids, sel)
    mask = torch.zeros((B, N, 1), dtype=torch.int64, device="cuda")
    depth = torch.zeros((B, N), dtype=torch.int32, device="cuda")
    ctx.tree_mask_build(parents, mask, depth)
    path = torch.zeros((B, N), dtype=torch.int32, device="cuda")
    alen = torch.zeros(B, dtype=torch.int32, device="cuda")
    bonus = torch.zeros(B, dtype=torch.int32, device="cuda")
    # acceptance on the reranked tree with its own tokens (the candidates' tokens, not fresh draws)
    ctx.accept_sampled(ids, parents, f32(s["p_target"]), f32(s["p_draft"]), f32(s["u_accept"]), f32(s["u_bonus"]),
                       path, alen, bonus)
    torch.cuda.synchronize()
    assert ctx.status_poll() == 0
    assert np.array_equal(parents.cpu().numpy(), want_parents) and np.array_equal(ids.cpu().numpy(), want_ids)
    wm, wd, ok = oracle.tree_mask(want_parents)
    assert ok and np.array_equal(gu.u64_host(mask), wm) and np.array_equal(depth.cpu().numpy(), wd) and wd.max() <= 3
    wp, wl, wb, _ = oracle.accept_sampled(want_ids, want_parents, s["p_target"], s["p_draft"], s["u_accept"], s["u_bonus"])
    assert np.array_equal(path.cpu().numpy(), wp) and np.array_equal(alen.cpu().numpy(), wl)
    assert np.array_equal(bonus.cpu().numpy(), wb)
    ctx.close()


def test_rerank_host_errors():
    from paper_2509_15235_b200 import binding
    ctx = binding.VerifyContext(2, 8, 4, 4, 64, 256, 1)
    i32 = lambda *shape: torch.zeros(shape, dtype=torch.int32, device="cuda")
    f32 = lambda *shape: torch.zeros(shape, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.VispecError):                        # K + 1 nodes exceed the context's tree size
        ctx.tree_rerank(i32(2, 20), i32(2, 20), f32(2, 20), 8, i32(2, 9), i32(2, 9), i32(2, 8))
    with pytest.raises(binding.VispecError):                        # K > M
        ctx.tree_rerank(i32(2, 3), i32(2, 3), f32(2, 3), 4, i32(2, 5), i32(2, 5), i32(2, 4))
    with pytest.raises(binding.VispecError):                        # M beyond the kernel's shared-memory table
        ctx.tree_rerank(i32(2, 2049), i32(2, 2049), f32(2, 2049), 4, i32(2, 5), i32(2, 5), i32(2, 4))
    ctx.close()
