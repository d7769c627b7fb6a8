"""GPU parity of the sampled (temperature > 0) acceptance against the fp64 oracle, through the C ABI.

Both sides decide in fp64 on the same fp32 inputs and the same uniforms, so path, length and bonus token are
compared for equality.  (The two differ in summation order only; a uniform would have to fall within ~1e-15 of
a threshold for a decision to flip, which the seeded inputs here do not do.)"""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_15235_b200 import synth

pytestmark = pytest.mark.gpu


def _run(parents, ids, p, ph, ua, ub):
    from paper_2509_15235_b200 import binding
    import gpu_util as gu
    B, N, V = p.shape
    ctx = binding.VerifyContext(max(B, 1), N, 4, 4, 64, 256, 1)
    f32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    path = torch.full((B, N), -9, dtype=torch.int32, device="cuda")
    alen = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    bonus = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    ctx.accept_sampled(gu.i32_dev(ids), gu.i32_dev(parents), f32(p), f32(ph), f32(ua), f32(ub), path, alen, bonus)
    torch.cuda.synchronize()
    status = ctx.status_poll()
    ctx.close()
    return path.cpu().numpy(), alen.cpu().numpy(), bonus.cpu().numpy(), status


def _check(parents, ids, p, ph, ua, ub, want_status=0):
    got = _run(parents, ids, p, ph, ua, ub)
    want = oracle.accept_sampled(ids, parents, p, ph, ua, ub)
    assert np.array_equal(got[1], want[1]), (got[1], want[1])
    assert np.array_equal(got[0], want[0])
    assert np.array_equal(got[2], want[2]), (got[2], want[2])
    assert got[3] == want_status
    return want


@pytest.mark.parametrize("name", ["tiny", "llava7b", "qwen7b", "llava13b_b4", "paper_tree"])
def test_sampled_acceptance_matches_the_oracle_on_the_workload_shapes(name):
    cfg = synth.get_config(name)
    t = synth.make_tree_inputs(cfg)
    for rep in range(3):
        s = synth.make_sampled_inputs(t["parents"], cfg.vocab, 7000 + 13 * cfg.config_id + rep)
        path, alen, bonus, bad = _check(t["parents"], s["draft_ids"], s["p_target"], s["p_draft"], s["u_accept"],
                                        s["u_bonus"])
        assert bad == 0 and np.all(bonus >= 0) and np.all(alen >= 1)


@pytest.mark.parametrize("V", [1, 2, 3, 5, 64, 127, 1000, 4099, 8191, 8192, 8196, 8197, 20001])
def test_sampled_acceptance_vocabulary_sizes_ragged_slices_and_many_rounds(V):
    """Small and odd vocabularies (scalar loads, slices that end early, empty warps and CTAs), flat distributions
    that reject often (many residual rounds per node), batches of 24 trees of 25 nodes."""
    rng = np.random.Generator(np.random.Philox(V))
    B, N = 24, 25
    parents = np.stack([synth.draw_tree(N, 4, 0, rng) for _ in range(B)])
    s = synth.make_sampled_inputs(parents, V, 100 + V, sharpness=1.0, disagreement=1.5)
    path, alen, bonus, bad = _check(parents, s["draft_ids"], s["p_target"], s["p_draft"], s["u_accept"], s["u_bonus"])
    assert bad == 0
    if V >= 64:
        assert (alen > 1).any() and (alen == 1).any()


def test_sampled_acceptance_degenerate_rows():
    """Zero entries, one-hot rows, an unnormalised target row whose residual is empty after the first rejection
    (the bonus token then comes from the target row), a target row without any weight (bonus -1), a star and a
    chain."""
    rng = np.random.Generator(np.random.Philox(99))
    V, N = 8200, 6
    star = np.array([-1, 0, 0, 0, 0, 0], dtype=np.int32)
    chain = np.arange(-1, N - 1, dtype=np.int32)
    parents = np.stack([star, chain, star, star, chain, star])
    B = parents.shape[0]
    s = synth.make_sampled_inputs(parents, V, 4242, sharpness=2.0)
    p, ph, ids = s["p_target"], s["p_draft"], s["draft_ids"]
    ua, ub = s["u_accept"], s["u_bonus"]
    p[0][:, rng.integers(0, V, size=V // 2)] = 0.0                 # sparse target rows
    ph[1] = 0.0                                                     # one-hot draft rows on the drafted tokens
    for i in range(N - 1):
        ph[1, i, ids[1, i + 1]] = 1.0
    p[2] = 0.5 * ph[2]; ua[2] = 0.75                                # ratio 1/2 everywhere, rejected, empty residual
    p[3] = 0.0                                                      # nothing to draw: bonus -1
    ua[3] = 0.5
    ua[5] = 0.999999                                                # every child of the star rejected: five rounds
    path, alen, bonus, bad = _check(parents, ids, p, ph, ua, ub)
    assert bad == 0 and alen[2] == 1 and bonus[2] >= 0 and bonus[3] == -1 and alen[3] == 1


def test_sampled_acceptance_flags_malformed_sequences():
    V, N = 50, 4
    rng = np.random.Generator(np.random.Philox(3))
    parents = np.array([[-1, 0, 1, 1], [-1, 0, 3, 1], [-1, 0, 0, 2], [0, 0, 1, 2]], dtype=np.int32)
    s = synth.make_sampled_inputs(np.array([[-1, 0, 1, 1]] * 4, dtype=np.int32), V, 5)
    ids = s["draft_ids"].copy()
    ids[2, 3] = V                                                   # token out of range
    got = _run(parents, ids, s["p_target"], s["p_draft"], s["u_accept"], s["u_bonus"])
    want = oracle.accept_sampled(ids, parents, s["p_target"], s["p_draft"], s["u_accept"], s["u_bonus"])
    assert want[3] == 3 and got[3] in (-8, -4)                      # BAD_TREE or RANGE, whichever block came first
    assert np.array_equal(got[0], want[0]) and np.array_equal(got[1], want[1]) and np.array_equal(got[2], want[2])
    assert list(got[1][1:]) == [0, 0, 0]


def test_sampled_acceptance_host_errors_and_empty_batch():
    from paper_2509_15235_b200 import binding
    ctx = binding.VerifyContext(2, 4, 4, 4, 64, 256, 1)
    i32 = lambda *shape: torch.zeros(shape, dtype=torch.int32, device="cuda")
    f32 = lambda *shape: torch.zeros(shape, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.VispecError):                        # more sequences than the context allows
        ctx.accept_sampled(i32(3, 4), i32(3, 4), f32(3, 4, 8), f32(3, 4, 8), f32(3, 4), f32(3), i32(3, 4), i32(3), i32(3))
    with pytest.raises(binding.VispecError):                        # rows not 16-byte aligned
        ctx.accept_sampled(i32(2, 4), i32(2, 4), f32(2 * 4 * 8 + 1)[1:].view(2, 4, 8), f32(2, 4, 8), f32(2, 4), f32(2),
                           i32(2, 4), i32(2), i32(2))
    before = ctx.launch_count()
    rc = ctx.lib.vispec_accept_sampled(ctx.handle, i32(2, 4).data_ptr(), i32(2, 4).data_ptr(), f32(2, 4, 8).data_ptr(),
                                       f32(2, 4, 8).data_ptr(), f32(2, 4).data_ptr(), f32(2).data_ptr(), 0, 4, 8,
                                       i32(2, 4).data_ptr(), i32(2).data_ptr(), i32(2).data_ptr(), None)
    assert rc == 0 and ctx.launch_count() == before
    ctx.close()
