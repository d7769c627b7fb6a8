"""GPU parity of the verification attention against the fp64 oracle, through the C ABI.

Tolerance: max-abs 2e-2 on bf16 outputs of O(1) magnitude (fp32 accumulation, probabilities and
outputs rounded to bf16: relative 2^-8 each); lse within 2e-3."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2509_15235_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 2e-2
LSE_TOL = 2e-3


@pytest.fixture(scope="module")
def gu():
    import gpu_util
    return gpu_util


def _check(gu, q, k, v, kv_len, mask, scale, split_form=0):
    out, lse, status = gu.run_attn(q, k, v, kv_len, mask, scale, split_form=split_form)
    want, want_lse = oracle.tree_attn(q, k, v, kv_len, mask, scale)
    assert status == 0
    assert not np.isnan(out).any()
    err = np.abs(out - want).max()
    assert err <= TOL, f"max abs err {err}"
    finite = np.isfinite(want_lse)
    assert np.array_equal(np.isfinite(lse), finite)
    if finite.any():
        assert np.abs(lse[finite] - want_lse[finite]).max() <= LSE_TOL
    return err


def _case(cfg, layer=0, S_max=None):
    t = synth.make_tree_inputs(cfg)
    x = synth.make_layer_tensors(cfg, layer, S_max=S_max)
    mask, _, _ = oracle.tree_mask(t["parents"])
    return x["q"], x["k_cache"], x["v_cache"], t["kv_len"], mask


def test_tiny_config_full_parity(gu):
    cfg = synth.get_config("tiny")
    _check(gu, *_case(cfg), 1 / math.sqrt(cfg.D))


@pytest.mark.parametrize("Hq,Hkv,D,N,S,S_max", [
    (4, 4, 64, 8, 256, 320),      # tiny-like
    (4, 4, 128, 60, 707, 832),    # MHA, ragged tail, several tiles
    (14, 2, 128, 60, 533, 640),   # GQA ratio 7 (Qwen2.5-VL-7B-like)
    (16, 2, 128, 16, 300, 384),   # GQA ratio 8, small tree
    (8, 1, 128, 128, 200, 384),   # GQA ratio 8, largest tree: 1024 query rows per kv head
    (2, 2, 64, 1, 77, 128),       # a single node (plain decode step)
    (4, 2, 128, 31, 1000, 1088),  # the paper's 30-token tree plus root
    (3, 3, 128, 65, 130, 256),    # two mask words
])
@pytest.mark.parametrize("split_form", [0, 1, 2, 3])
def test_shapes_span_tiles_tails_and_group_sizes(gu, Hq, Hkv, D, N, S, S_max, split_form):
    rng = np.random.Generator(np.random.Philox(Hq * 1000 + N))
    B = 2
    q = synth.normal_bf16((B, N, Hq, D), 1 + N)
    k = synth.normal_bf16((B, Hkv, S_max, D), 2 + N)
    v = synth.normal_bf16((B, Hkv, S_max, D), 3 + N)
    kv_len = np.array([S, max(0, S - 61)], dtype=np.int32)
    parents = np.stack([synth.draw_tree(N, 6, 4, rng) for _ in range(B)])
    mask, _, _ = oracle.tree_mask(parents)
    _check(gu, q, k, v, kv_len, mask, 1 / math.sqrt(D), split_form=split_form)


def test_arbitrary_mask_bits_all_ones_and_zero_rows(gu):
    B, N, Hq, Hkv, D, S_max = 2, 20, 4, 2, 128, 256
    q = synth.normal_bf16((B, N, Hq, D), 21); k = synth.normal_bf16((B, Hkv, S_max, D), 22)
    v = synth.normal_bf16((B, Hkv, S_max, D), 23)
    rng = np.random.default_rng(9)
    mask = rng.integers(0, 1 << 20, size=(B, N, 1), dtype=np.int64).astype(np.uint64)
    mask[0, 3, 0] = (1 << 20) - 1          # all ones
    mask[1, 5, 0] = 0                      # no tree key at all
    _check(gu, q, k, v, np.array([100, 0], dtype=np.int32), mask, 0.11)


def test_empty_allowed_set_gives_zero_and_minus_inf(gu):
    B, N, Hq, Hkv, D, S_max = 1, 4, 2, 2, 64, 64
    q = synth.normal_bf16((B, N, Hq, D), 31); k = synth.normal_bf16((B, Hkv, S_max, D), 32)
    v = synth.normal_bf16((B, Hkv, S_max, D), 33)
    mask = np.array([[[0], [2], [0], [8]]], dtype=np.uint64)
    out, lse, status = gu.run_attn(q, k, v, np.array([0], dtype=np.int32), mask, 0.5)
    want, want_lse = oracle.tree_attn(q, k, v, [0], mask, 0.5)
    assert status == 0 and (out[0, 0] == 0).all() and (out[0, 2] == 0).all()
    assert np.isneginf(lse[0, :, 0]).all() and np.isneginf(lse[0, :, 2]).all()
    assert np.abs(out - want).max() <= TOL


def test_slots_past_the_tree_may_hold_nan_patterns(gu):
    cfg = synth.get_config("tiny")
    q, k, v, kv_len, mask = _case(cfg, S_max=384)
    k = k.copy(); v = v.copy()
    end = int(kv_len[0]) + cfg.N
    k[:, :, end:] = 0x7FC0; v[:, :, end:] = 0x7FC0
    k[:, :, end + 3] = 0x7F80; v[:, :, end + 3] = 0xFF80      # +inf / -inf
    _check(gu, q, k, v, kv_len, mask, 0.125)


def test_non_ancestor_rows_do_not_influence_a_node(gu):
    """Hidden tree rows get weight exactly 0, so replacing them by other finite rows leaves a node's
    output bit-identical (a NaN there would not: 0 * NaN; hidden rows hold finite data by contract)."""
    B, N, Hq, Hkv, D, S_max = 1, 12, 2, 1, 128, 128
    rng = np.random.Generator(np.random.Philox(77))
    q = synth.normal_bf16((B, N, Hq, D), 41); k = synth.normal_bf16((B, Hkv, S_max, D), 42)
    v = synth.normal_bf16((B, Hkv, S_max, D), 43)
    parents = synth.draw_tree(N, 3, 3, rng)[None]
    mask, _, _ = oracle.tree_mask(parents)
    S = 50
    base, _, _ = gu.run_attn(q, k, v, [S], mask, 0.1)
    i = N - 1
    k2, v2 = k.copy(), v.copy()
    for t in range(N):
        if not (int(mask[0, i, 0]) >> t) & 1:
            k2[0, :, S + t] = k[0, :, (t * 7) % S]; v2[0, :, S + t] = 0x42C8   # other finite rows (v = 100)
    out2, _, _ = gu.run_attn(q, k2, v2, [S], mask, 0.1)
    assert np.array_equal(out2[0, i], base[0, i])


def test_large_scores_stay_finite(gu):
    """Scores of magnitude ~1e3: the running-max rescale must keep everything finite."""
    B, N, Hq, Hkv, D, S_max = 1, 8, 2, 2, 64, 192
    q = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(synth.normal_bf16((B, N, Hq, D), 51)) * 30)
    k = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(synth.normal_bf16((B, Hkv, S_max, D), 52)) * 30)
    v = synth.normal_bf16((B, Hkv, S_max, D), 53)
    mask, _, _ = oracle.tree_mask(np.arange(-1, N - 1, dtype=np.int32)[None])
    out, lse, _ = gu.run_attn(q, k, v, [150], mask, 0.125)
    want, want_lse = oracle.tree_attn(q, k, v, [150], mask, 0.125)
    assert np.isfinite(out).all() and np.abs(out - want).max() <= TOL
    assert np.abs(lse - want_lse).max() <= 2e-3 * np.abs(want_lse).max()


def test_overlong_sequence_is_zeroed_with_status(gu):
    B, N, Hq, Hkv, D, S_max = 2, 8, 2, 2, 64, 128
    q = synth.normal_bf16((B, N, Hq, D), 61); k = synth.normal_bf16((B, Hkv, S_max, D), 62)
    v = synth.normal_bf16((B, Hkv, S_max, D), 63)
    mask, _, _ = oracle.tree_mask(np.tile(np.arange(-1, N - 1, dtype=np.int32), (B, 1)))
    out, lse, status = gu.run_attn(q, k, v, [125, 100], mask, 0.125)
    assert status == -4 and (out[0] == 0).all()
    want, _ = oracle.tree_attn(q[1:], k[1:], v[1:], [100], mask[1:], 0.125)
    assert np.abs(out[1] - want[0]).max() <= TOL


def test_host_side_argument_errors(gu):
    from paper_2509_15235_b200 import binding
    ctx = binding.VerifyContext(1, 8, 2, 2, 64, 128, 2)
    q = torch.zeros((1, 8, 2, 64), dtype=torch.bfloat16, device="cuda")
    kv_len = torch.zeros(1, dtype=torch.int32, device="cuda")
    mask = torch.zeros((1, 8, 1), dtype=torch.int64, device="cuda")
    with pytest.raises(binding.VispecError) as e:
        ctx.tree_verify_attn(0, q, kv_len, mask, 1.0, q.clone())
    assert e.value.code == -9                                    # nothing registered
    cache = torch.zeros((1, 2, 128, 64), dtype=torch.bfloat16, device="cuda")
    ctx.cache_register(0, cache, cache.clone())
    with pytest.raises(binding.VispecError) as e:
        ctx.tree_verify_attn(2, q, kv_len, mask, 1.0, q.clone())
    assert e.value.code == -4                                    # layer out of range
    with pytest.raises(binding.VispecError) as e:
        ctx.tree_verify_attn(0, q, kv_len, mask, 1.0, q.clone(), k_cache=cache.clone())
    assert e.value.code == -9                                    # not the registered pointer
    big = torch.zeros((1, 9, 2, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.VispecError) as e:
        ctx.tree_verify_attn(0, big, kv_len, mask, 1.0, big.clone())
    assert e.value.code == -3                                    # N > N_max
    ctx.tree_verify_attn(0, q, kv_len, mask, 1.0, q.clone(), k_cache=cache)
    torch.cuda.synchronize()


@pytest.mark.parametrize("split_form", [0, 1, 2])
@pytest.mark.parametrize("name", ["llava7b", "qwen7b"])
def test_full_size_layer_parity(gu, name, split_form):
    """One whole layer at benchmark size, every output element against the oracle, for both ways of
    combining the pieces of a head (partials + merge kernel; clusters) and for the library's own choice (the
    launch configuration bench.py times; on qwen7b that is the layout with 64-row blocks, which the forced forms
    do not take)."""
    cfg = synth.get_config(name)
    _check(gu, *_case(cfg, layer=1), 1 / math.sqrt(cfg.D), split_form=split_form)


def test_full_size_batched_variable_length_parity(gu):
    cfg = synth.get_config("llava13b_b4")
    q, k, v, kv_len, mask = _case(cfg, layer=0)
    # the oracle on 4 x 40 heads x ~4000 keys takes a while: check 8 heads of every sequence
    heads = [0, 5, 13, 21, 27, 33, 38, 39]
    out, lse, status = gu.run_attn(q, k, v, kv_len, mask, 1 / math.sqrt(cfg.D))
    assert status == 0 and not np.isnan(out).any()
    want, want_lse = oracle.tree_attn(q[:, :, heads], k[:, heads], v[:, heads], kv_len, mask, 1 / math.sqrt(cfg.D))
    assert np.abs(out[:, :, heads] - want).max() <= TOL
    assert np.abs(lse[:, heads] - want_lse).max() <= LSE_TOL
    # and every one of the 40 heads of the longest sequence
    b = int(np.argmax(kv_len))
    want, want_lse = oracle.tree_attn(q[b:b + 1], k[b:b + 1], v[b:b + 1], kv_len[b:b + 1], mask[b:b + 1], 1 / math.sqrt(cfg.D))
    assert np.abs(out[b:b + 1] - want).max() <= TOL
    assert np.abs(lse[b:b + 1] - want_lse).max() <= LSE_TOL


@pytest.mark.parametrize("name", ["qwen3b_S2048_N16_B1", "qwen3b_S8192_N60_B4", "qwen3b_S32768_N128_B1",
                                  "qwen3b_S16384_N16_B8"])
def test_long_response_sweep_cells(gu, name):
    """Sweep cells at full size: the whole GPU result is produced, and the oracle recomputes every
    output of one kv head's group (heads are independent, so this samples the result exactly)."""
    cfg = synth.get_config(name)
    q, k, v, kv_len, mask = _case(cfg)
    scale = 1 / math.sqrt(cfg.D)
    out, lse, status = gu.run_attn(q, k, v, kv_len, mask, scale)
    assert status == 0 and not np.isnan(out).any()
    kvh = cfg.Hkv - 1
    hs = slice(kvh * cfg.G, (kvh + 1) * cfg.G)
    want, want_lse = oracle.tree_attn(q[:, :, hs], k[:, kvh:kvh + 1], v[:, kvh:kvh + 1], kv_len, mask, scale)
    assert np.abs(out[:, :, hs] - want).max() <= TOL
    assert np.abs(lse[:, hs] - want_lse).max() <= LSE_TOL


def test_options_and_fallbacks_give_the_same_attention(gu):
    """Early prefix prefetch off, more sequences than the tensor-core kernel takes per call (generic kernel),
    and a non-positive scale (generic kernel: the maximum no longer commutes with the scale)."""
    from paper_2509_15235_b200 import binding
    rng = np.random.Generator(np.random.Philox(2024))
    Hq, Hkv, D, N, S_max = 4, 2, 128, 12, 384
    for B, scale, early in ((2, 0.09, 0), (33, 0.09, None), (2, 0.0, None), (2, -0.05, None)):
        q = synth.normal_bf16((B, N, Hq, D), 71 + B); k = synth.normal_bf16((B, Hkv, S_max, D), 72 + B)
        v = synth.normal_bf16((B, Hkv, S_max, D), 73 + B)
        kv_len = rng.integers(0, S_max - N, size=B).astype(np.int32)
        parents = np.stack([synth.draw_tree(N, 4, 3, rng) for _ in range(B)])
        mask, _, _ = oracle.tree_mask(parents)
        out, lse, status = gu.run_attn(q, k, v, kv_len, mask, scale, early_prefetch=early)
        want, want_lse = oracle.tree_attn(q, k, v, kv_len, mask, scale)
        assert status == 0
        assert np.abs(out - want).max() <= TOL
        assert np.abs(lse - want_lse).max() <= LSE_TOL
    ctx = binding.VerifyContext(1, 8, 2, 2, 64, 128, 1)
    with pytest.raises(binding.VispecError) as e:
        ctx.ctx_set_option(99, 1)
    assert e.value.code == -5
    with pytest.raises(binding.VispecError) as e:
        ctx.ctx_set_option(binding.OPT_SPLIT_FORM, 7)
    assert e.value.code == -4


def test_redundant_image_keys_stress_the_softmax(gu):
    """Sec. 4.1 of the paper: image tokens are highly redundant, identical tokens get identical scores (Eq. 2)
    and their softmax mass is spread evenly (Eq. 3-4).  1296 identical 'image' keys followed by ordinary text
    keys: a huge, flat block of probability mass, against the oracle; and with every key identical the output
    must be the mean of the visible V rows (Eq. 4), checked directly."""
    B, N, Hq, Hkv, D, S, S_max = 1, 16, 4, 2, 128, 1500, 1664
    rng = np.random.Generator(np.random.Philox(404))
    q = synth.normal_bf16((B, N, Hq, D), 81); k = synth.normal_bf16((B, Hkv, S_max, D), 82)
    v = synth.normal_bf16((B, Hkv, S_max, D), 83)
    k[:, :, :1296] = k[:, :, :1]                       # the image span repeats one key per head
    parents = synth.draw_tree(N, 4, 3, rng)[None]
    mask, _, _ = oracle.tree_mask(parents)
    _check(gu, q, k, v, np.array([S], dtype=np.int32), mask, 1 / math.sqrt(D))
    k[:, :, :] = k[:, :, :1]                           # every key identical: weights are uniform over the visible set
    out, lse, status = gu.run_attn(q, k, v, [S], mask, 1 / math.sqrt(D))
    assert status == 0
    vf = synth.bf16_bits_to_f32(v).astype(np.float64)
    for i in range(N):
        vis = list(range(S)) + [S + t for t in range(N) if (int(mask[0, i, 0]) >> t) & 1]
        for h in range(Hq):
            assert np.abs(out[0, i, h] - vf[0, h // (Hq // Hkv), vis].mean(axis=0)).max() <= TOL


def test_stream_probe_runs_and_validates_its_arguments(gu):
    """The measurement aid: it only reads, so the check is that it runs clean on ragged lengths (including a
    rejected sequence, which it skips) and that the host-side validation answers."""
    from paper_2509_15235_b200 import binding
    ctx = binding.VerifyContext(3, 60, 4, 2, 128, 1024, 2)
    k = torch.zeros((3, 2, 1024, 128), dtype=torch.bfloat16, device="cuda")
    ctx.cache_register(0, k, k.clone())
    ctx.stream_probe(0, gu.i32_dev([900, 0, 1000]), 60)        # 1000 + 60 > 1024: skipped
    torch.cuda.synchronize()
    assert ctx.status_poll() == 0
    with pytest.raises(binding.VispecError) as e:
        ctx.stream_probe(1, gu.i32_dev([1, 2, 3]), 60)
    assert e.value.code == -9                                   # layer 1 has no registered cache
    ctx64 = binding.VerifyContext(1, 8, 2, 2, 64, 128, 1)
    c = torch.zeros((1, 2, 128, 64), dtype=torch.bfloat16, device="cuda")
    ctx64.cache_register(0, c, c.clone())
    with pytest.raises(binding.VispecError) as e:
        ctx64.stream_probe(0, gu.i32_dev([10]), 8)
    assert e.value.code == -5                                   # D = 64: no TMA maps


def test_seeded_random_shapes_against_the_oracle(gu):
    """Sixty seeded draws of (batch, heads, group size, tree size, lengths, split form): every output element
    against the oracle.  Lengths straddle tile boundaries; some sequences are empty."""
    rng = np.random.Generator(np.random.Philox(2024))
    for case in range(60):
        B = int(rng.integers(1, 6))
        Hkv = int(rng.choice([1, 2, 3, 4, 8]))
        G = int(rng.choice([1, 2, 4, 7, 8]))
        N = int(rng.choice([1, 2, 7, 16, 31, 60, 64, 65, 100, 128]))
        S_hi = int(rng.choice([0, 5, 127, 128, 129, 400, 1000, 1400]))
        kv_len = rng.integers(0, S_hi + 1, size=B).astype(np.int32)
        S_max = (int(kv_len.max()) + N + 127) // 128 * 128 + int(rng.choice([0, 128]))
        split_form = int(rng.integers(0, 4))
        q = synth.normal_bf16((B, N, Hkv * G, 128), 9000 + 3 * case)
        k = synth.normal_bf16((B, Hkv, S_max, 128), 9001 + 3 * case)
        v = synth.normal_bf16((B, Hkv, S_max, 128), 9002 + 3 * case)
        parents = np.stack([synth.draw_tree(N, 8, 0, rng) for _ in range(B)])
        mask, _, _ = oracle.tree_mask(parents)
        _check(gu, q, k, v, kv_len, mask, 1 / math.sqrt(128), split_form=split_form)
