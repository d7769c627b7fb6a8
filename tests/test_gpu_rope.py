"""GPU parity of the rotary embedding / tree-row placement against the fp64 oracle, through the C ABI.

Both sides form the angle and the rotation in fp64 and round once to bf16, so the results agree bit for bit
except where the fp64 value sits within a few fp64 ulps of a bf16 rounding boundary (the two sincos routines
and a fused multiply-add may differ in the last place).  The bar: v rows and every untouched cache slot
bit-exact; rotated values identical on at least 99.99 % of the elements and never more than one bf16 step apart."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_15235_b200 import synth

pytestmark = pytest.mark.gpu


def _ordered(bits):
    """bf16 bit patterns -> integers whose order is the order of the values (so a difference counts steps)."""
    b = bits.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b)


def _run(B, N, Hq, Hkv, D, S_max, kv_len, positions, theta, seed, layers=2, layer=1):
    from paper_2509_15235_b200 import binding
    import gpu_util as gu
    q = synth.normal_bf16((B, N, Hq, D), seed); k = synth.normal_bf16((B, N, Hkv, D), seed + 1)
    v = synth.normal_bf16((B, N, Hkv, D), seed + 2)
    kc = synth.normal_bf16((B, Hkv, S_max, D), seed + 3); vc = synth.normal_bf16((B, Hkv, S_max, D), seed + 4)
    ctx = binding.VerifyContext(max(B, 1), N, Hq, Hkv, D, S_max, layers)
    kd, vd, qd = gu.bf16_dev(kc), gu.bf16_dev(vc), gu.bf16_dev(q)
    ctx.cache_register(layer, kd, vd)
    ctx.rope_tree_rows(layer, qd, gu.bf16_dev(k), gu.bf16_dev(v), gu.i32_dev(positions), gu.i32_dev(kv_len), theta)
    torch.cuda.synchronize()
    status = ctx.status_poll()
    got = gu.bf16_bits(qd), gu.bf16_bits(kd), gu.bf16_bits(vd)
    ctx.close()
    want = oracle.rope_rows(q, k, v, positions, kv_len, kc, vc, theta)
    return got, want, status


def _compare(got, want):
    gq, gk, gv = got
    wq, wk, wv, _ = want
    assert np.array_equal(gv, wv)                               # copies and untouched slots: exact
    for g, w in ((gq, wq), (gk, wk)):
        step = np.abs(_ordered(g) - _ordered(w))
        assert step.max() <= 1
        assert (step != 0).mean() <= 1e-4


@pytest.mark.parametrize("name", ["tiny", "llava7b", "qwen7b", "paper_tree"])
def test_rope_rows_match_the_oracle_on_the_workload_shapes(name):
    cfg = synth.get_config(name)
    t = synth.make_tree_inputs(cfg)
    _, depth, _ = oracle.tree_mask(t["parents"])
    S_max = min(cfg.S_max, int(t["kv_len"].max()) + cfg.N + 5)   # a short cache: placement is all that is checked of it
    positions = (t["kv_len"][:, None] + depth).astype(np.int32)
    theta = 1e6 if name.startswith("qwen") else 1e4
    got, want, status = _run(cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D, S_max, t["kv_len"], positions, theta, 500)
    assert status == 0 and want[3] == 0
    _compare(got, want)


def test_rope_rows_edges_full_cache_one_node_large_positions_and_a_skipped_sequence():
    from paper_2509_15235_b200 import binding
    # N = 1, kv_len + N == S_max exactly, positions up to 131071, D = 64
    kv_len = np.array([31, 0, 17], dtype=np.int32)
    positions = np.array([[131071], [0], [40000]], dtype=np.int32)
    got, want, status = _run(3, 1, 4, 2, 64, 32, kv_len, positions, 1e6, 900, layers=1, layer=0)
    assert status == 0
    _compare(got, want)
    # one sequence does not fit: skipped on both sides, reported in the status word, the others are done
    kv_len = np.array([4, 30, 9], dtype=np.int32)
    positions = np.tile(np.arange(5, dtype=np.int32), (3, 1)) + kv_len[:, None]
    got, want, status = _run(3, 5, 8, 8, 128, 32, kv_len, positions, 1e4, 901, layers=1, layer=0)
    assert want[3] == 1 and status == -4
    _compare(got, want)


def test_rope_rows_host_errors_and_empty_batch():
    from paper_2509_15235_b200 import binding
    import gpu_util as gu
    ctx = binding.VerifyContext(2, 4, 4, 2, 64, 64, 1)
    q = torch.zeros((2, 4, 4, 64), dtype=torch.bfloat16, device="cuda")
    kn = torch.zeros((2, 4, 2, 64), dtype=torch.bfloat16, device="cuda")
    pos = torch.zeros((2, 4), dtype=torch.int32, device="cuda")
    kvl = torch.zeros(2, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.VispecError):                     # nothing registered for the layer
        ctx.rope_tree_rows(0, q, kn, kn, pos, kvl, 1e4)
    kc = torch.zeros((2, 2, 64, 64), dtype=torch.bfloat16, device="cuda")
    ctx.cache_register(0, kc, kc.clone())
    with pytest.raises(binding.VispecError):                     # layer out of range
        ctx.rope_tree_rows(1, q, kn, kn, pos, kvl, 1e4)
    with pytest.raises(binding.VispecError):                     # base must exceed 1
        ctx.rope_tree_rows(0, q, kn, kn, pos, kvl, 1.0)
    before = ctx.launch_count()
    import ctypes
    rc = ctx.lib.vispec_rope_tree_rows(ctx.handle, 0, q.data_ptr(), kn.data_ptr(), kn.data_ptr(), pos.data_ptr(),
                                       kvl.data_ptr(), 0, 4, ctypes.c_float(1e4), None)   # empty batch: no launch
    assert rc == 0
    assert ctx.launch_count() == before
    ctx.rope_tree_rows(0, q, kn, kn, pos, kvl, 1e4)
    torch.cuda.synchronize()
    assert ctx.launch_count() == before + 1 and ctx.status_poll() == 0
    ctx.close()


@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (8, 2)])
def test_commit_then_rope_then_attention_chained_on_one_stream(Hq, Hkv):
    """The end of one cycle and the start of the next, enqueued back to back with nothing in between:
    vispec_accept_commit writes the new kv_len and commits rows, vispec_rope_tree_rows places the next tree's rows behind
    the new length, vispec_tree_verify_attn (early prefix reads on) takes that same device kv_len.  The attention must
    see the committed length and rows; everything against the oracle's chain."""
    from paper_2509_15235_b200 import binding
    import gpu_util as gu
    B, N, D, S_max = 2, 24, 128, 1792
    rng = np.random.Generator(np.random.Philox(31 + Hq))
    scale = 1.0 / np.sqrt(D)
    for rep in range(4):
        kv_len = np.array([1500 + 7 * rep, 901 - 3 * rep], dtype=np.int32)
        kc = synth.normal_bf16((B, Hkv, S_max, D), 700 + rep); vc = synth.normal_bf16((B, Hkv, S_max, D), 710 + rep)
        parents1 = np.stack([synth.draw_tree(N, 6, 4, rng) for _ in range(B)])
        target = rng.integers(0, 50, size=(B, N)).astype(np.int32)
        draft = np.where(rng.random((B, N)) < 0.8, np.take_along_axis(target, np.maximum(parents1, 0), 1),
                         rng.integers(50, 99, size=(B, N))).astype(np.int32)
        parents2 = np.stack([synth.draw_tree(N, 6, 4, rng) for _ in range(B)])
        q2 = synth.normal_bf16((B, N, Hq, D), 720 + rep)
        k2 = synth.normal_bf16((B, N, Hkv, D), 730 + rep); v2 = synth.normal_bf16((B, N, Hkv, D), 740 + rep)
        # the oracle's chain
        o_path, o_len, _ = oracle.accept(draft, target, parents1)
        o_k, o_v, o_new = oracle.kv_compact(kc, vc, o_path, o_len, kv_len)
        mask2, depth2, _ = oracle.tree_mask(parents2)
        positions2 = (o_new[:, None] + depth2).astype(np.int32)
        o_q, o_k2, o_v2, skipped = oracle.rope_rows(q2, k2, v2, positions2, o_new, o_k, o_v, 1e4)
        assert skipped == 0
        want, want_lse = oracle.tree_attn(o_q, o_k2, o_v2, o_new, mask2, scale)
        # the same chain on one stream, no host involvement between the calls
        ctx = binding.VerifyContext(B, N, Hq, Hkv, D, S_max, 1)
        kd, vd = gu.bf16_dev(kc), gu.bf16_dev(vc)
        ctx.cache_register(0, kd, vd)
        qd, k2d, v2d = gu.bf16_dev(q2), gu.bf16_dev(k2), gu.bf16_dev(v2)
        path = torch.zeros((B, N), dtype=torch.int32, device="cuda")
        alen = torch.zeros(B, dtype=torch.int32, device="cuda"); bonus = torch.zeros_like(alen)
        new_len = torch.zeros_like(alen)
        out = torch.full((B, N, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((B, Hq, N), float("nan"), dtype=torch.float32, device="cuda")
        args = (gu.i32_dev(draft), gu.i32_dev(target), gu.i32_dev(parents1), gu.i32_dev(kv_len), gu.i32_dev(positions2),
                gu.u64_dev(mask2))
        torch.cuda.synchronize()
        ctx.accept_commit(0, 1, args[0], args[1], args[2], args[3], path, alen, bonus, new_len)
        ctx.rope_tree_rows(0, qd, k2d, v2d, args[4], new_len, 1e4)
        ctx.tree_verify_attn(0, qd, new_len, args[5], scale, out, lse)
        torch.cuda.synchronize()
        assert ctx.status_poll() == 0
        assert np.array_equal(new_len.cpu().numpy(), o_new)
        assert np.abs(out.float().cpu().numpy() - want).max() <= 2e-2
        assert np.abs(lse.cpu().numpy() - want_lse).max() <= 2e-3
        ctx.close()


@pytest.mark.parametrize("split_form", [0, 1, 2, 3])
@pytest.mark.parametrize("B,N,Hq,Hkv,kv_len,S_max", [
    (1, 60, 8, 8, [1100], 1280),            # one row block per head, several tiles, tree rows inside one tile
    (2, 60, 4, 4, [1000, 350], 1152),       # tree rows straddle a tile boundary (1000 + 60 > 1024); two sequences
    (2, 60, 14, 2, [533, 472], 640),        # 7 query heads per kv head: four row blocks share the tree rows
    (1, 31, 8, 2, [97], 256),               # the paper's tree; the first tile already holds tree rows
])
def test_fused_rope_attention_matches_rope_then_attention_of_the_oracle(B, N, Hq, Hkv, kv_len, S_max, split_form):
    """vispec_tree_verify_attn_rope against oracle.rope_rows followed by oracle.tree_attn: the cache afterwards (v rows and
    untouched slots bit-exact, rotated k rows within one bf16 step on at most 1e-4 of the elements), q untouched, and
    the attention output within its tolerance."""
    from paper_2509_15235_b200 import binding
    import gpu_util as gu
    D = 128
    rng = np.random.Generator(np.random.Philox(900 + N + Hq))
    kv_len = np.asarray(kv_len, dtype=np.int32)
    q = synth.normal_bf16((B, N, Hq, D), 801); k = synth.normal_bf16((B, N, Hkv, D), 802)
    v = synth.normal_bf16((B, N, Hkv, D), 803)
    kc = synth.normal_bf16((B, Hkv, S_max, D), 804); vc = synth.normal_bf16((B, Hkv, S_max, D), 805)
    parents = np.stack([synth.draw_tree(N, 6, 4, rng) for _ in range(B)])
    mask, depth, _ = oracle.tree_mask(parents)
    positions = (kv_len[:, None] + depth).astype(np.int32)
    theta, scale = 1e6, 1.0 / np.sqrt(D)
    o_q, o_k, o_v, skipped = oracle.rope_rows(q, k, v, positions, kv_len, kc, vc, theta)
    assert skipped == 0
    want, want_lse = oracle.tree_attn(o_q, o_k, o_v, kv_len, mask, scale)

    ctx = binding.VerifyContext(B, N, Hq, Hkv, D, S_max, 1)
    if split_form:
        ctx.ctx_set_option(binding.OPT_SPLIT_FORM, split_form)
    kd, vd, qd = gu.bf16_dev(kc), gu.bf16_dev(vc), gu.bf16_dev(q)
    ctx.cache_register(0, kd, vd)
    table = ctx.rope_table_build(gu.i32_dev(positions), theta)
    out = torch.full((B, N, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, Hq, N), float("nan"), dtype=torch.float32, device="cuda")
    ctx.tree_verify_attn_rope(0, qd, gu.bf16_dev(k), gu.bf16_dev(v), table, gu.i32_dev(kv_len), gu.u64_dev(mask), scale, out, lse)
    torch.cuda.synchronize()
    assert ctx.status_poll() == 0
    assert np.array_equal(gu.bf16_bits(qd), q)                      # q is read only
    assert np.array_equal(gu.bf16_bits(vd), o_v)                    # copies and untouched slots: exact
    step = np.abs(_ordered(gu.bf16_bits(kd)) - _ordered(o_k))
    assert step.max() <= 1 and (step != 0).mean() <= 1e-4
    assert np.abs(out.float().cpu().numpy() - want).max() <= 2e-2
    assert np.abs(lse.cpu().numpy() - want_lse).max() <= 2e-3
    ctx.close()


@pytest.mark.parametrize("split_form", [0, 1])
def test_fused_rope_attention_leaves_a_sequence_that_does_not_fit_alone(split_form):
    """kv_len + N > S_max for one sequence: its cache rows stay as they were (nothing is written past its slots), its
    output is zero with lse = -inf, the status word says so, and the other sequence is served as usual."""
    from paper_2509_15235_b200 import binding
    import gpu_util as gu
    B, N, Hq, Hkv, D, S_max = 2, 24, 4, 4, 128, 512
    kv_len = np.array([S_max - N + 3, 300], dtype=np.int32)           # sequence 0 would need 3 slots beyond its cache
    rng = np.random.Generator(np.random.Philox(977))
    q = synth.normal_bf16((B, N, Hq, D), 811); k = synth.normal_bf16((B, N, Hkv, D), 812)
    v = synth.normal_bf16((B, N, Hkv, D), 813)
    kc = synth.normal_bf16((B, Hkv, S_max, D), 814); vc = synth.normal_bf16((B, Hkv, S_max, D), 815)
    parents = np.stack([synth.draw_tree(N, 5, 3, rng) for _ in range(B)])
    mask, depth, _ = oracle.tree_mask(parents)
    positions = (kv_len[:, None] + depth).astype(np.int32)
    theta, scale = 1e4, 1.0 / np.sqrt(D)
    o_q, o_k, o_v, skipped = oracle.rope_rows(q, k, v, positions, kv_len, kc, vc, theta)
    assert skipped == 1
    want, want_lse = oracle.tree_attn(o_q[1:], o_k[1:], o_v[1:], kv_len[1:], mask[1:], scale)

    ctx = binding.VerifyContext(B, N, Hq, Hkv, D, S_max, 1)
    if split_form:
        ctx.ctx_set_option(binding.OPT_SPLIT_FORM, split_form)
    # the caches sit in the middle of one allocation whose margins must come back untouched as well
    pad = 64 * D
    kbuf = torch.full((B * Hkv * S_max * D + 2 * pad,), 1.5, dtype=torch.bfloat16, device="cuda")
    vbuf = torch.full_like(kbuf, 2.5)
    kd = kbuf[pad:-pad].view(B, Hkv, S_max, D); vd = vbuf[pad:-pad].view(B, Hkv, S_max, D)
    kd.copy_(gu.bf16_dev(kc)); vd.copy_(gu.bf16_dev(vc))
    ctx.cache_register(0, kd, vd)
    table = ctx.rope_table_build(gu.i32_dev(positions), theta)
    out = torch.full((B, N, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, Hq, N), float("nan"), dtype=torch.float32, device="cuda")
    ctx.tree_verify_attn_rope(0, gu.bf16_dev(q), gu.bf16_dev(k), gu.bf16_dev(v), table, gu.i32_dev(kv_len), gu.u64_dev(mask),
                              scale, out, lse)
    torch.cuda.synchronize()
    assert ctx.status_poll() == -4
    assert (kbuf[:pad] == 1.5).all() and (kbuf[-pad:] == 1.5).all() and (vbuf[:pad] == 2.5).all() and (vbuf[-pad:] == 2.5).all()
    assert np.array_equal(gu.bf16_bits(kd[0].contiguous()), kc[0]) and np.array_equal(gu.bf16_bits(vd[0].contiguous()), vc[0])
    assert np.array_equal(gu.bf16_bits(vd[1].contiguous()), o_v[1])
    o = out.float().cpu().numpy()
    assert (o[0] == 0).all() and np.isneginf(lse[0].cpu().numpy()).all()
    assert np.abs(o[1] - want[0]).max() <= 2e-2
    assert np.abs(lse[1].cpu().numpy() - want_lse[0]).max() <= 2e-3
    ctx.close()


def test_fused_rope_attention_refuses_what_it_does_not_serve():
    from paper_2509_15235_b200 import binding
    ctx = binding.VerifyContext(1, 8, 2, 2, 64, 128, 1)            # head size 64: the generic kernel's territory
    c = torch.zeros((1, 2, 128, 64), dtype=torch.bfloat16, device="cuda")
    ctx.cache_register(0, c, c.clone())
    q = torch.zeros((1, 8, 2, 64), dtype=torch.bfloat16, device="cuda")
    pos = torch.zeros((1, 8), dtype=torch.int32, device="cuda")
    table = ctx.rope_table_build(pos, 1e4)
    with pytest.raises(binding.VispecError) as e:
        ctx.tree_verify_attn_rope(0, q, q.clone(), q.clone(), table, pos[:, 0].contiguous(),
                                  torch.ones((1, 8, 1), dtype=torch.int64, device="cuda"), 0.1, q.clone())
    assert e.value.code == -5
    with pytest.raises(binding.VispecError):
        ctx.rope_table_build(pos, 1.0)
    ctx.close()
