"""Paged cache: the attention and the commit on a block pool + block table give what the contiguous calls give.

Paging is a layout, not arithmetic: the oracle runs on the contiguous cache the pool was cut from.  The paged
attention must agree with the oracle within the attention tolerance AND bit for bit with the contiguous GPU call
(same tiles, same order of operations)."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2509_15235_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 2e-2
LSE_TOL = 2e-3
NAN = np.uint16(0x7FC0)


def _page(cache, page_rows, rng, spare=3):
    """[B,Hkv,S_max,D] -> (pool [num_blocks,Hkv,page_rows,D] with unused blocks NaN, table [B, S_max/page_rows])."""
    B, Hkv, S_max, D = cache[0].shape
    per = S_max // page_rows
    nb = B * per + spare
    perm = rng.permutation(nb)[:B * per].reshape(B, per).astype(np.int32)
    pools = []
    for c in cache:
        pool = np.full((nb, Hkv, page_rows, D), NAN, dtype=np.uint16)
        blocks = c.reshape(B, Hkv, per, page_rows, D).transpose(0, 2, 1, 3, 4)          # [B, per, Hkv, rows, D]
        pool[perm.reshape(-1)] = blocks.reshape(B * per, Hkv, page_rows, D)
        pools.append(pool)
    return pools, perm


def _unpage(pool, table, S_max):
    B, per = table.shape
    nb, Hkv, rows, D = pool.shape
    blocks = pool[table.reshape(-1)].reshape(B, per, Hkv, rows, D).transpose(0, 2, 1, 3, 4)
    return blocks.reshape(B, Hkv, per * rows, D)[:, :, :S_max]


def _run_paged(q, pools, table, kv_len, mask, scale, split_form=0, N_max=None, token_major=False):
    from paper_2509_15235_b200 import binding
    import gpu_util as gu
    B, N, Hq, D = q.shape
    nb, Hkv, rows, _ = pools[0].shape
    ctx = binding.VerifyContext(max(B, 1), N_max or N, Hq, Hkv, D, table.shape[1] * rows, 1)
    if split_form:
        ctx.ctx_set_option(binding.OPT_SPLIT_FORM, split_form)
    if token_major:
        pools = [np.ascontiguousarray(x.transpose(0, 2, 1, 3)) for x in pools]
    kd, vd = gu.bf16_dev(pools[0]), gu.bf16_dev(pools[1])
    ctx.cache_register_paged(0, kd, vd, token_major)
    out = torch.full((B, N, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, Hq, N), float("nan"), dtype=torch.float32, device="cuda")
    ctx.tree_verify_attn_paged(0, gu.bf16_dev(q), gu.i32_dev(kv_len), gu.i32_dev(table), gu.u64_dev(mask), scale, out, lse)
    torch.cuda.synchronize()
    status = ctx.status_poll()
    ctx.close()
    return out.float().cpu().numpy(), lse.cpu().numpy(), status


def _case(B, N, Hq, Hkv, S_list, S_max, seed):
    rng = np.random.Generator(np.random.Philox(seed))
    D = 128
    q = synth.normal_bf16((B, N, Hq, D), seed + 1)
    k = synth.normal_bf16((B, Hkv, S_max, D), seed + 2)
    v = synth.normal_bf16((B, Hkv, S_max, D), seed + 3)
    kv_len = np.array(S_list, dtype=np.int32)
    parents = np.stack([synth.draw_tree(N, 6, 4, rng) for _ in range(B)])
    mask, _, _ = oracle.tree_mask(parents)
    return q, k, v, kv_len, mask, rng


@pytest.mark.parametrize("page_rows", [16, 32, 64, 128])
@pytest.mark.parametrize("split_form", [0, 1, 2, 3])
@pytest.mark.parametrize("token_major", [False, True])
def test_paged_attention_equals_contiguous_and_oracle(page_rows, split_form, token_major):
    import gpu_util as gu
    B, N, Hq, Hkv, S_max = 3, 60, 8, 2, 1152
    q, k, v, kv_len, mask, rng = _case(B, N, Hq, Hkv, [1000, 707, 3], S_max, 100 + page_rows)
    scale = 1 / math.sqrt(128)
    pools, table = _page((k, v), page_rows, rng)
    # entries of blocks that start at or past kv_len + N must never be read: poison them
    table = table.copy()
    for b in range(B):
        first_unused = -(-(int(kv_len[b]) + N) // page_rows)
        table[b, first_unused:] = 2 ** 30
    out, lse, status = _run_paged(q, pools, table, kv_len, mask, scale, split_form, token_major=token_major)
    assert status == 0 and not np.isnan(out).any()
    want, want_lse = oracle.tree_attn(q, k, v, kv_len, mask, scale)
    assert np.abs(out - want).max() <= TOL and np.abs(lse - want_lse).max() <= LSE_TOL
    ref, ref_lse, st = gu.run_attn(q, k, v, kv_len, mask, scale, split_form=split_form)
    assert st == 0 and np.array_equal(out, ref) and np.array_equal(lse, ref_lse)


@pytest.mark.parametrize("B,N,Hq,Hkv,S_list,S_max,page_rows,token_major", [
    (2, 128, 8, 1, [200, 77], 384, 32, False),       # largest tree: 1024 query rows per kv head, two mask words
    (2, 1, 4, 2, [129, 0], 256, 16, True),           # a single node (plain decode step); an empty prefix
    (32, 9, 2, 2, list(range(3, 35)), 128, 64, False),   # the most sequences a call takes
    (3, 65, 3, 3, [130, 64, 1], 256, 128, True),     # two mask words with one head per kv head
])
def test_paged_attention_edge_shapes(B, N, Hq, Hkv, S_list, S_max, page_rows, token_major):
    q, k, v, kv_len, mask, rng = _case(B, N, Hq, Hkv, S_list, S_max, 500 + B + N)
    pools, table = _page((k, v), page_rows, rng)
    scale = 1 / math.sqrt(128)
    out, lse, status = _run_paged(q, pools, table, kv_len, mask, scale, token_major=token_major)
    want, want_lse = oracle.tree_attn(q, k, v, kv_len, mask, scale)
    assert status == 0 and not np.isnan(out).any()
    assert np.abs(out - want).max() <= TOL
    finite = np.isfinite(want_lse)
    assert np.array_equal(np.isfinite(lse), finite) and np.abs(lse[finite] - want_lse[finite]).max() <= LSE_TOL


def test_paged_attention_rows_past_the_end_may_hold_anything():
    B, N, Hq, Hkv, S_max = 2, 31, 4, 4, 512
    q, k, v, kv_len, mask, rng = _case(B, N, Hq, Hkv, [300, 129], S_max, 7)
    for b in range(B):
        k[b, :, kv_len[b] + N:] = NAN
        v[b, :, kv_len[b] + N:] = NAN
    pools, table = _page((k, v), 32, rng)
    out, lse, status = _run_paged(q, pools, table, kv_len, mask, 0.09)
    want, want_lse = oracle.tree_attn(q, k, v, kv_len, mask, 0.09)
    assert status == 0 and not np.isnan(out).any()
    assert np.abs(out - want).max() <= TOL and np.abs(lse - want_lse).max() <= LSE_TOL


def test_paged_attention_full_size_llava7b_layer():
    cfg = synth.get_config("llava7b")
    t = synth.make_tree_inputs(cfg)
    x = synth.make_layer_tensors(cfg, 0)
    mask, _, _ = oracle.tree_mask(t["parents"])
    rng = np.random.Generator(np.random.Philox(11))
    pools, table = _page((x["k_cache"], x["v_cache"]), 16, rng, spare=17)
    scale = 1 / math.sqrt(cfg.D)
    out, lse, status = _run_paged(x["q"], pools, table, t["kv_len"], mask, scale)
    want, want_lse = oracle.tree_attn(x["q"], x["k_cache"], x["v_cache"], t["kv_len"], mask, scale)
    assert status == 0
    assert np.abs(out - want).max() <= TOL and np.abs(lse - want_lse).max() <= LSE_TOL


def test_paged_attention_skips_what_does_not_fit_and_flags_bad_entries():
    B, N, Hq, Hkv, S_max = 2, 16, 4, 2, 256
    q, k, v, kv_len, mask, rng = _case(B, N, Hq, Hkv, [200, 250], S_max, 9)      # 250 + 16 > 256: skipped
    pools, table = _page((k, v), 64, rng)
    out, lse, status = _run_paged(q, pools, table, kv_len, mask, 0.09)
    want, want_lse = oracle.tree_attn(q, k, v, np.array([200, 0], np.int32), mask, 0.09)
    assert status == -4
    assert np.abs(out[0] - want[0]).max() <= TOL and np.all(out[1] == 0) and np.all(np.isneginf(lse[1]))
    # a table entry outside the pool: reported, read as zeros, nothing else disturbed
    kv_len = np.array([200, 100], dtype=np.int32)
    bad = table.copy(); bad[1, 0] = pools[0].shape[0] + 5
    out, lse, status = _run_paged(q, pools, bad, kv_len, mask, 0.09)
    k2, v2 = k.copy(), v.copy(); k2[1, :, :64] = 0; v2[1, :, :64] = 0
    want, want_lse = oracle.tree_attn(q, k2, v2, kv_len, mask, 0.09)
    assert status == -4 and np.abs(out - want).max() <= TOL


def test_paged_commit_matches_the_oracle_on_the_logical_cache():
    from paper_2509_15235_b200 import binding
    import gpu_util as gu
    B, N, Hkv, D, S_max, layers, rows = 3, 12, 2, 128, 256, 2, 16
    rng = np.random.Generator(np.random.Philox(21))
    path = np.full((B, N), -1, dtype=np.int32)
    path[0, :4] = [0, 2, 5, 11]; path[1, :1] = [0]; path[2, :6] = [0, 1, 2, 3, 9, 10]
    alen = np.array([4, 1, 6], dtype=np.int32)
    kv_len = np.array([100, 0, 244], dtype=np.int32)              # 244 + 12 == 256: the last slots of the table
    ctx = binding.VerifyContext(B, N, 4, Hkv, D, S_max, layers)
    caches, pools_d, tables = [], [], None
    perm_rng = np.random.Generator(np.random.Philox(22))
    for l in range(layers):
        k = rng.integers(0, 65536, size=(B, Hkv, S_max, D), dtype=np.int64).astype(np.uint16)
        v = rng.integers(0, 65536, size=(B, Hkv, S_max, D), dtype=np.int64).astype(np.uint16)
        pools, table = _page((k, v), rows, np.random.Generator(np.random.Philox(22)))   # one table for all layers
        tables = table
        kd, vd = gu.bf16_dev(pools[0]), gu.bf16_dev(pools[1])
        ctx.cache_register_paged(l, kd, vd)
        caches.append((k, v)); pools_d.append((kd, vd, pools))
    out_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.kv_compact_paged(0, layers, gu.i32_dev(path), gu.i32_dev(alen), gu.i32_dev(kv_len), gu.i32_dev(tables), out_len)
    torch.cuda.synchronize()
    assert ctx.status_poll() == 0
    for l in range(layers):
        wk, wv, wl = oracle.kv_compact(caches[l][0], caches[l][1], path, alen, kv_len)
        gk, gv = gu.bf16_bits(pools_d[l][0]), gu.bf16_bits(pools_d[l][1])
        assert np.array_equal(_unpage(gk, tables, S_max), wk) and np.array_equal(_unpage(gv, tables, S_max), wv)
        unused = np.setdiff1d(np.arange(gk.shape[0]), tables.reshape(-1))
        assert np.array_equal(gk[unused], pools_d[l][2][0][unused])                    # blocks outside the table untouched
        assert np.array_equal(out_len.cpu().numpy(), wl)
    # contiguous calls refuse a paged layer and the other way round
    with pytest.raises(binding.VispecError):
        ctx.kv_compact(0, layers, gu.i32_dev(path), gu.i32_dev(alen), gu.i32_dev(kv_len), out_len)
    ctx.close()


@pytest.mark.parametrize("token_major", [False, True])
def test_paged_accept_commit_and_rope_match_the_oracle(token_major):
    from paper_2509_15235_b200 import binding
    import gpu_util as gu
    cfg = synth.get_config("paper_tree")
    B, N, Hq, Hkv, D, layers, rows, S_max = 3, cfg.N, 8, 2, 128, 2, 32, 512
    rng = np.random.Generator(np.random.Philox(31))
    parents = np.stack([synth.draw_tree(N, 3, 8, rng) for _ in range(B)])
    ids = [synth.draw_ids(parents[b], 1000, 0.7, rng) for b in range(B)]
    draft = np.stack([d for d, _ in ids]); target = np.stack([t for _, t in ids])
    kv_len = np.array([100, 0, S_max - N], dtype=np.int32)
    _, depth, _ = oracle.tree_mask(parents)
    positions = (kv_len[:, None] + depth).astype(np.int32)
    ctx = binding.VerifyContext(B, N, Hq, Hkv, D, S_max, layers)
    state, table = [], None
    for l in range(layers):
        k = synth.normal_bf16((B, Hkv, S_max, D), 300 + l); v = synth.normal_bf16((B, Hkv, S_max, D), 310 + l)
        pools, table = _page((k, v), rows, np.random.Generator(np.random.Philox(32)))
        if token_major:
            pools = [np.ascontiguousarray(x.transpose(0, 2, 1, 3)) for x in pools]
        kd, vd = gu.bf16_dev(pools[0]), gu.bf16_dev(pools[1])
        ctx.cache_register_paged(l, kd, vd, token_major)
        state.append([k, v, kd, vd])
    tab_d = gu.i32_dev(table)
    pool_bits = (lambda t: gu.bf16_bits(t).transpose(0, 2, 1, 3)) if token_major else gu.bf16_bits   # back to [block, head, slot, D]
    # RoPE + placement on every layer, then acceptance + commit over both layers in one launch
    for l in range(layers):
        q = synth.normal_bf16((B, N, Hq, D), 320 + l); kn = synth.normal_bf16((B, N, Hkv, D), 330 + l)
        vn = synth.normal_bf16((B, N, Hkv, D), 340 + l)
        qd = gu.bf16_dev(q)
        ctx.rope_tree_rows_paged(l, qd, gu.bf16_dev(kn), gu.bf16_dev(vn), gu.i32_dev(positions), gu.i32_dev(kv_len), tab_d, 1e4)
        wq, wk, wv, skipped = oracle.rope_rows(q, kn, vn, positions, kv_len, state[l][0], state[l][1], 1e4)
        assert skipped == 0
        torch.cuda.synchronize()
        gk = _unpage(pool_bits(state[l][2]), table, S_max); gv = _unpage(pool_bits(state[l][3]), table, S_max)
        assert np.array_equal(gv, wv)
        step = np.abs(gk.astype(np.int32) - wk.astype(np.int32))          # bit patterns of equal sign: steps
        assert step.max() <= 1 and (step != 0).mean() <= 1e-4
        assert np.abs(gu.bf16_bits(qd).astype(np.int32) - wq.astype(np.int32)).max() <= 1
        state[l][0], state[l][1] = gk, gv                                  # the commit below starts from what the GPU holds
    path = torch.zeros((B, N), dtype=torch.int32, device="cuda")
    alen = torch.zeros(B, dtype=torch.int32, device="cuda"); bonus = torch.zeros(B, dtype=torch.int32, device="cuda")
    new_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.accept_commit_paged(0, layers, gu.i32_dev(draft), gu.i32_dev(target), gu.i32_dev(parents), gu.i32_dev(kv_len),
                            tab_d, path, alen, bonus, new_len)
    torch.cuda.synchronize()
    assert ctx.status_poll() == 0
    wp, wl, wb = oracle.accept(draft, target, parents)
    assert np.array_equal(path.cpu().numpy(), wp) and np.array_equal(alen.cpu().numpy(), wl)
    assert np.array_equal(bonus.cpu().numpy(), wb) and (wl > 1).any()
    for l in range(layers):
        wk, wv, wn = oracle.kv_compact(state[l][0], state[l][1], wp, wl, kv_len)
        assert np.array_equal(_unpage(pool_bits(state[l][2]), table, S_max), wk)
        assert np.array_equal(_unpage(pool_bits(state[l][3]), table, S_max), wv)
        assert np.array_equal(new_len.cpu().numpy(), wn)
    ctx.close()


def test_paged_host_errors():
    from paper_2509_15235_b200 import binding
    ctx = binding.VerifyContext(2, 8, 4, 2, 128, 256, 2)
    pool = torch.zeros((10, 2, 16, 128), dtype=torch.bfloat16, device="cuda")
    odd = torch.zeros((10, 2, 24, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.VispecError):                        # page size not one of 16/32/64/128
        ctx.cache_register_paged(0, odd, odd)
    ctx.cache_register_paged(0, pool, pool.clone())
    cont = torch.zeros((2, 2, 256, 128), dtype=torch.bfloat16, device="cuda")
    ctx.cache_register(1, cont, cont.clone())
    q = torch.zeros((2, 8, 4, 128), dtype=torch.bfloat16, device="cuda")
    kvl = torch.zeros(2, dtype=torch.int32, device="cuda")
    tab = torch.zeros((2, 16), dtype=torch.int32, device="cuda")
    mask = torch.zeros((2, 8, 1), dtype=torch.int64, device="cuda")
    with pytest.raises(binding.VispecError):                        # contiguous layer through the paged call
        ctx.tree_verify_attn_paged(1, q, kvl, tab, mask, 0.1, torch.empty_like(q))
    with pytest.raises(binding.VispecError):                        # paged layer through the contiguous call
        ctx.tree_verify_attn(0, q, kvl, mask, 0.1, torch.empty_like(q))
    ctx.close()
    ctx64 = binding.VerifyContext(1, 8, 4, 4, 64, 256, 1)
    p64 = torch.zeros((10, 4, 16, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.VispecError):                        # D = 64 has no paged path
        ctx64.cache_register_paged(0, p64, p64.clone())
    ctx64.close()
