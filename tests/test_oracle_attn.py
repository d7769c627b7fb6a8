"""Pins for the attention oracle (Eq. 1 restricted to prefix + ancestors).

Witnesses that are not the oracle: torch's causal scaled-dot-product attention in fp64 (chain
tree), a numpy matmul softmax (all-ones mask), the closed forms of Eq. 3 and Eq. 4, and
invariants of softmax attention."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2509_15235_b200 import synth


def _f64(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def _bits(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _rand_case(seed, B=2, N=9, Hq=4, Hkv=2, D=16, S_max=48):
    rng = np.random.Generator(np.random.Philox(seed))
    q = synth.normal_bf16((B, N, Hq, D), seed * 10 + 1)
    k = synth.normal_bf16((B, Hkv, S_max, D), seed * 10 + 2)
    v = synth.normal_bf16((B, Hkv, S_max, D), seed * 10 + 3)
    kv_len = rng.integers(0, S_max - N + 1, size=B).astype(np.int32)
    parents = np.stack([synth.draw_tree(N, 4, 3, rng) for _ in range(B)])
    return q, k, v, kv_len, parents


def _chain_mask(B, N):
    return oracle.tree_mask(np.tile(np.arange(-1, N - 1, dtype=np.int32), (B, 1)))[0]


def _ones_mask(B, N):
    W = (N + 63) // 64
    m = np.zeros((B, N, W), dtype=np.uint64)
    for t in range(N):
        m[:, :, t // 64] |= np.uint64(1) << np.uint64(t % 64)
    return m


@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (4, 2), (6, 1)])
def test_chain_tree_equals_causal_attention_from_torch(Hq, Hkv):
    B, N, D, S_max = 2, 7, 16, 40
    q, k, v, kv_len, _ = _rand_case(3, B, N, Hq, Hkv, D, S_max)
    kv_len[:] = [20, 33]
    scale = 1 / math.sqrt(D)
    out, _ = oracle.tree_attn(q, k, v, kv_len, _chain_mask(B, N), scale)
    G = Hq // Hkv
    for b in range(B):
        S = int(kv_len[b]); T = S + N
        K = torch.from_numpy(_f64(k[b, :, :T])).repeat_interleave(G, dim=0)     # [Hq,T,D]
        V = torch.from_numpy(_f64(v[b, :, :T])).repeat_interleave(G, dim=0)
        Q = torch.zeros(Hq, T, D, dtype=torch.float64)
        Q[:, S:] = torch.from_numpy(_f64(q[b])).permute(1, 0, 2)
        ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V, is_causal=True, scale=scale)
        ref = ref[:, S:].permute(1, 0, 2).numpy()                                   # [N,Hq,D]
        assert np.abs(out[b] - ref).max() < 1e-12


def test_all_ones_mask_equals_dense_attention_numpy():
    B, N, Hq, Hkv, D, S_max = 2, 9, 4, 2, 16, 48
    q, k, v, kv_len, _ = _rand_case(4, B, N, Hq, Hkv, D, S_max)
    scale = 0.37
    out, lse = oracle.tree_attn(q, k, v, kv_len, _ones_mask(B, N), scale)
    for b in range(B):
        T = int(kv_len[b]) + N
        for h in range(Hq):
            Kh = _f64(k[b, h // 2, :T]); Vh = _f64(v[b, h // 2, :T]); Qh = _f64(q[b, :, h])
            s = scale * Qh @ Kh.T
            p = np.exp(s - s.max(axis=1, keepdims=True))
            ref = (p / p.sum(axis=1, keepdims=True)) @ Vh
            assert np.abs(out[b, :, h] - ref).max() < 1e-12
            ref_lse = np.log(np.exp(s).sum(axis=1))
            assert np.abs(lse[b, h] - ref_lse).max() < 1e-12


def test_random_tree_equals_numpy_masked_attention():
    """A dense [N, S+N] boolean mask built with the recurrence, applied in numpy."""
    B, N, Hq, Hkv, D, S_max = 2, 9, 4, 2, 16, 48
    q, k, v, kv_len, parents = _rand_case(5, B, N, Hq, Hkv, D, S_max)
    mask = oracle.tree_mask(parents)[0]
    out, _ = oracle.tree_attn(q, k, v, kv_len, mask, 0.25)
    for b in range(B):
        S = int(kv_len[b]); T = S + N
        allow = np.zeros((N, T), dtype=bool)
        allow[:, :S] = True
        for i in range(N):
            a = i
            while a != -1:
                allow[i, S + a] = True
                a = int(parents[b, a])
        for h in range(Hq):
            s = 0.25 * _f64(q[b, :, h]) @ _f64(k[b, h // 2, :T]).T
            s = np.where(allow, s, -np.inf)
            p = np.exp(s - s.max(axis=1, keepdims=True))
            ref = (p / p.sum(axis=1, keepdims=True)) @ _f64(v[b, h // 2, :T])
            assert np.abs(out[b, :, h] - ref).max() < 1e-12


def test_identical_keys_give_the_mean_of_allowed_values_eq4():
    """Eq. 4: when all keys coincide every weight is 1/R and the output is the mean of V."""
    B, N, Hq, Hkv, D, S_max = 1, 5, 2, 1, 8, 32
    q = synth.normal_bf16((B, N, Hq, D), 11)
    key = synth.normal_bf16((D,), 12)
    k = np.broadcast_to(key, (B, Hkv, S_max, D)).copy()
    v = synth.normal_bf16((B, Hkv, S_max, D), 13)
    parents = np.array([[-1, 0, 0, 1, 2]], dtype=np.int32)
    mask = oracle.tree_mask(parents)[0]
    S = 20
    out, lse = oracle.tree_attn(q, k, v, [S], mask, 1 / math.sqrt(D))
    anc = {0: [0], 1: [0, 1], 2: [0, 2], 3: [0, 1, 3], 4: [0, 2, 4]}
    V = _f64(v[0, 0])
    for i in range(N):
        rows = list(range(S)) + [S + a for a in anc[i]]
        assert np.abs(out[0, i, :, :] - V[rows].mean(axis=0)).max() < 1e-13
        score = (1 / math.sqrt(D)) * (_f64(q[0, i]) @ _f64(key))
        assert np.abs(lse[0, :, i] - (score + math.log(len(rows)))).max() < 1e-12


@pytest.mark.parametrize("R", [1, 7, 100, 3000])
def test_unique_key_weight_matches_eq3(R):
    """Eq. 3: R identical keys with score A and one unique key with score B give the unique key
    the weight e^B / (R e^A + e^B).  The value rows are chosen so the output *is* that weight."""
    D = 8
    qv = np.zeros(D); qv[0] = 2.0; qv[1] = 1.0          # q
    s_key = np.zeros(D); s_key[0] = 0.5                  # redundant key  -> A = scale * 1.0
    t_key = np.zeros(D); t_key[0] = 1.5; t_key[1] = -0.25  # unique key   -> B = scale * 2.75
    scale = 0.5
    A, Bs = scale * 1.0, scale * 2.75
    S = R + 1
    S_max = S + 1
    k = np.tile(_bits(s_key), (1, 1, S_max, 1))
    u = R // 2                                           # the unique key sits inside the run
    k[0, 0, u] = _bits(t_key)
    v = np.zeros((1, 1, S_max, D), dtype=np.uint16)
    v[0, 0, u, 0] = _bits([1.0])[0]                      # out[0] = alpha_u
    v[0, 0, :S, 1] = _bits([1.0])[0]                     # out[1] = sum of all weights = 1 - alpha_root
    q = _bits(qv).reshape(1, 1, 1, D)
    mask = np.zeros((1, 1, 1), dtype=np.uint64)          # the root's own row is switched off
    out, lse = oracle.tree_attn(q, k, v, [S], mask, scale)
    want = math.exp(Bs) / (R * math.exp(A) + math.exp(Bs))
    assert abs(out[0, 0, 0, 0] - want) < 1e-12
    assert abs(out[0, 0, 0, 1] - 1.0) < 1e-12
    assert abs(lse[0, 0, 0] - math.log(R * math.exp(A) + math.exp(Bs))) < 1e-12


def test_softmax_invariants():
    B, N, Hq, Hkv, D, S_max = 1, 9, 4, 2, 16, 48
    q, k, v, kv_len, parents = _rand_case(6, B, N, Hq, Hkv, D, S_max)
    kv_len[:] = 25
    S = 25
    mask = oracle.tree_mask(parents)[0]
    scale = 0.25
    out, lse = oracle.tree_attn(q, k, v, kv_len, mask, scale)
    # outputs are convex combinations of the value rows
    Vf = _f64(v[0, :, :S + N])
    for h in range(Hq):
        lo, hi = Vf[h // 2].min(axis=0), Vf[h // 2].max(axis=0)
        assert (out[0, :, h] >= lo - 1e-12).all() and (out[0, :, h] <= hi + 1e-12).all()
    # permuting the committed prefix changes nothing
    perm = np.random.default_rng(0).permutation(S)
    k2, v2 = k.copy(), v.copy()
    k2[:, :, :S] = k[:, :, perm]; v2[:, :, :S] = v[:, :, perm]
    out2, lse2 = oracle.tree_attn(q, k2, v2, kv_len, mask, scale)
    assert np.abs(out2 - out).max() < 1e-13 and np.abs(lse2 - lse).max() < 1e-12
    # a node never sees a non-ancestor: changing that row leaves its output bit-identical
    i = N - 1
    non_anc = [t for t in range(N) if not (int(mask[0, i, 0]) >> t) & 1]
    assert non_anc
    k3, v3 = k.copy(), v.copy()
    for t in non_anc:
        k3[0, :, S + t] ^= 0x1234; v3[0, :, S + t] ^= 0x0321
    out3, _ = oracle.tree_attn(q, k3, v3, kv_len, mask, scale)
    assert np.array_equal(out3[0, i], out[0, i])
    # slots past kv_len + N are never read
    k4, v4 = k.copy(), v.copy()
    k4[:, :, S + N:] = 0x7FC0; v4[:, :, S + N:] = 0x7FC0          # NaN patterns
    out4, _ = oracle.tree_attn(q, k4, v4, kv_len, mask, scale)
    assert np.array_equal(out4, out)
    # GQA: heads of one group share K/V; swapping two query heads swaps the outputs
    q5 = q.copy(); q5[:, :, [0, 1]] = q[:, :, [1, 0]]
    out5, _ = oracle.tree_attn(q5, k, v, kv_len, mask, scale)
    assert np.array_equal(out5[:, :, 0], out[:, :, 1]) and np.array_equal(out5[:, :, 1], out[:, :, 0])


def test_score_shift_invariance_and_lse_shift():
    """Adding a vector c to every key shifts every score of row i by scale*<q_i,c>: outputs keep
    their value and lse moves by exactly that shift."""
    D = 8
    rng = np.random.default_rng(2)
    # small integers are exact in bf16 and keep every sum exact in fp64
    q = _bits(rng.integers(-3, 4, size=(1, 4, 2, D)).astype(np.float32))
    k = rng.integers(-3, 4, size=(1, 2, 24, D)).astype(np.float32)
    v = _bits(rng.integers(-8, 9, size=(1, 2, 24, D)).astype(np.float32))
    c = rng.integers(-2, 3, size=D).astype(np.float32)
    parents = np.array([[-1, 0, 1, 0]], dtype=np.int32)
    mask = oracle.tree_mask(parents)[0]
    out, lse = oracle.tree_attn(q, _bits(k), v, [16], mask, 0.125)
    out2, lse2 = oracle.tree_attn(q, _bits(k + c), v, [16], mask, 0.125)
    assert np.abs(out2 - out).max() < 1e-13
    shift = 0.125 * (_f64(q[0]) @ c.astype(np.float64))        # [N,Hq]
    assert np.abs((lse2 - lse)[0] - shift.T).max() < 1e-12


def test_split_kv_merge_by_lse_reproduces_one_pass():
    """Two disjoint key ranges attended separately and merged with
    out = (e^{l1} o1 + e^{l2} o2) / (e^{l1} + e^{l2}) equal the one-pass result: pins lse."""
    B, N, Hq, Hkv, D, S_max = 1, 6, 4, 2, 16, 64
    q, k, v, _, parents = _rand_case(7, B, N, Hq, Hkv, D, S_max)
    S, cut = 40, 17
    mask = oracle.tree_mask(parents)[0]
    scale = 0.3
    full, lse = oracle.tree_attn(q, k, v, [S], mask, scale)
    zero = np.zeros_like(mask)
    o1, l1 = oracle.tree_attn(q, k, v, [cut], zero, scale)               # keys [0, cut)
    o2, l2 = oracle.tree_attn(q, k[:, :, cut:], v[:, :, cut:], [S - cut], mask, scale)
    l1t, l2t = l1.transpose(0, 2, 1)[..., None], l2.transpose(0, 2, 1)[..., None]   # [B,N,Hq,1]
    m = np.maximum(l1t, l2t)
    w1, w2 = np.exp(l1t - m), np.exp(l2t - m)
    merged = (w1 * o1 + w2 * o2) / (w1 + w2)
    assert np.abs(merged - full).max() < 1e-12
    assert np.abs((m + np.log(w1 + w2))[..., 0].transpose(0, 2, 1) - lse).max() < 1e-12


def test_empty_allowed_set_gives_zero_and_minus_inf():
    q = synth.normal_bf16((1, 2, 1, 8), 1)
    k = synth.normal_bf16((1, 1, 8, 8), 2)
    v = synth.normal_bf16((1, 1, 8, 8), 3)
    mask = np.zeros((1, 2, 1), dtype=np.uint64)
    mask[0, 1, 0] = 2                                   # node 1 sees only itself, node 0 nothing
    out, lse = oracle.tree_attn(q, k, v, [0], mask, 1.0)
    assert (out[0, 0] == 0).all() and lse[0, 0, 0] == -np.inf
    assert np.abs(out[0, 1, 0] - _f64(v[0, 0, 1])).max() == 0 and np.isfinite(lse[0, 0, 1])


def test_oracle_rejects_overflowing_lengths():
    q = synth.normal_bf16((1, 4, 1, 8), 1)
    k = synth.normal_bf16((1, 1, 8, 8), 2)
    with pytest.raises(ValueError):
        oracle.tree_attn(q, k, k, [5], np.zeros((1, 4, 1), dtype=np.uint64), 1.0)


def test_bf16_helpers_round_to_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.1415927, 0.0], dtype=np.float32)
    bits = synth.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)
    big = np.random.default_rng(0).standard_normal(100000).astype(np.float32)
    ref = torch.from_numpy(big).to(torch.bfloat16)
    assert np.array_equal(synth.f32_to_bf16_bits(big), ref.view(torch.int16).numpy().view(np.uint16))
    assert np.array_equal(synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(big)), ref.float().numpy())
