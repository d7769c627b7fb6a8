"""Pins of the rotary-embedding oracle (CPU only): against what the mathematics fixes, not against itself.

The paper uses the target LLM unchanged (Sec. 3.2); LLaVA-v1.6 (Vicuna) and Qwen2.5-VL rotate q and k by
position with the half-split pairing.  Pins: position 0 is the identity; each pair is a plane rotation, written
here as a complex multiplication by exp(i*angle) in numpy; norms are preserved; the score of a rotated q against
a rotated k depends on the position difference only; placement touches exactly the slots kv_len + i."""
import numpy as np
import pytest

import oracle
from paper_2509_15235_b200 import synth


def _f(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def _case(B=2, N=5, Hq=4, Hkv=2, D=64, S_max=48, seed=11):
    q = synth.normal_bf16((B, N, Hq, D), seed); k = synth.normal_bf16((B, N, Hkv, D), seed + 1)
    v = synth.normal_bf16((B, N, Hkv, D), seed + 2)
    kc = synth.normal_bf16((B, Hkv, S_max, D), seed + 3); vc = synth.normal_bf16((B, Hkv, S_max, D), seed + 4)
    return q, k, v, kc, vc


def test_position_zero_is_the_identity_and_placement_touches_only_the_tree_slots():
    q, k, v, kc, vc = _case()
    B, N = q.shape[:2]
    kv_len = np.array([7, 30], dtype=np.int32)
    pos = np.zeros((B, N), dtype=np.int32)
    q2, kc2, vc2, skipped = oracle.rope_rows(q, k, v, pos, kv_len, kc, vc, 10000.0)
    assert skipped == 0 and np.array_equal(q2, q)
    for b in range(B):
        S = kv_len[b]
        assert np.array_equal(kc2[b, :, S:S + N], k[b].transpose(1, 0, 2))
        assert np.array_equal(vc2[b, :, S:S + N], v[b].transpose(1, 0, 2))
        keep = np.ones(kc.shape[2], dtype=bool); keep[S:S + N] = False
        assert np.array_equal(kc2[b][:, keep], kc[b][:, keep]) and np.array_equal(vc2[b][:, keep], vc[b][:, keep])


def test_each_pair_is_a_complex_rotation_by_position_times_inverse_frequency():
    q, k, v, kc, vc = _case(D=128)
    B, N, Hq, D = q.shape
    rng = np.random.default_rng(3)
    pos = rng.integers(0, 5000, size=(B, N)).astype(np.int32)
    theta = 1.0e6
    q2, kc2, _, _ = oracle.rope_rows(q, k, v, pos, np.array([3, 11], dtype=np.int32), kc, vc, theta)
    inv = theta ** (-2.0 * np.arange(D // 2) / D)
    rot = np.exp(1j * pos[:, :, None, None].astype(np.float64) * inv)          # [B,N,1,D/2]
    z = (_f(q)[..., :D // 2] + 1j * _f(q)[..., D // 2:]) * rot
    want = np.concatenate([z.real, z.imag], axis=-1)
    got = _f(q2)
    assert np.abs(got - want).max() <= 2.0 ** -8 * np.abs(want).max()           # one bf16 rounding
    # most elements are the correctly rounded value exactly
    assert np.mean(synth.f32_to_bf16_bits(want.astype(np.float32)) == q2) > 0.99
    zk = (_f(k)[..., :D // 2] + 1j * _f(k)[..., D // 2:]) * rot
    wk = np.concatenate([zk.real, zk.imag], axis=-1)                            # [B,N,Hkv,D]
    for b, S in enumerate((3, 11)):
        assert np.abs(_f(kc2[b, :, S:S + N]) - wk[b].transpose(1, 0, 2)).max() <= 2.0 ** -8 * np.abs(wk).max()


def test_rotation_keeps_norms_and_scores_depend_on_the_position_difference_only():
    B, N, H, D, S_max = 1, 2, 1, 64, 16
    q = synth.normal_bf16((B, N, H, D), 21); k = synth.normal_bf16((B, N, H, D), 22)
    q[0, 1] = q[0, 0]; k[0, 1] = k[0, 0]                                         # same vectors at two positions
    kc = np.zeros((B, H, S_max, D), dtype=np.uint16)
    scores = []
    for p0 in (5, 1234):
        pos = np.array([[p0, p0 + 17]], dtype=np.int32)
        q2, kc2, _, _ = oracle.rope_rows(q, k, k, pos, np.array([0], dtype=np.int32), kc, kc, 10000.0)
        assert np.abs(np.linalg.norm(_f(q2), axis=-1) - np.linalg.norm(_f(q), axis=-1)).max() <= 0.05
        # q at position p0 + 17 against k at position p0: difference 17 both times
        scores.append(float(_f(q2)[0, 1, 0] @ _f(kc2)[0, 0, 0]))
    assert abs(scores[0] - scores[1]) <= 0.02 * (abs(scores[0]) + 1.0)              # bf16 rounding of 64 terms


def test_out_of_range_sequence_is_skipped():
    q, k, v, kc, vc = _case()
    B, N = q.shape[:2]
    pos = np.ones((B, N), dtype=np.int32)
    q2, kc2, vc2, skipped = oracle.rope_rows(q, k, v, pos, np.array([44, 2], dtype=np.int32), kc, vc, 10000.0)   # 44 + 5 > 48
    assert skipped == 1
    assert np.array_equal(q2[0], q[0]) and np.array_equal(kc2[0], kc[0]) and np.array_equal(vc2[0], vc[0])
    assert not np.array_equal(q2[1], q[1])
