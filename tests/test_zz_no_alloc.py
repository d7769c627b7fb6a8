"""The allocation-free attention entry point against the regular one, through the C ABI.

vispec_tree_verify_attn_static serves callers that cannot allocate device memory when they run
(fixed memory pools, plugins without an allocator, streams that must not see cudaMalloc's implicit
synchronisation).  Its scratch is one array inside the library that every call shares and that keeps
the last call's contents, so the check runs two different problems back to back: the second must
not be disturbed by what the first left behind.  This file sorts last on purpose."""
import math

import numpy as np
import pytest
import torch

from paper_2509_15235_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 2e-2


def _problem(seed, B, N, Hq, Hkv, D, S_max, kv_len):
    import gpu_util as gu
    import oracle
    rng = np.random.Generator(np.random.Philox(seed))
    q = synth.normal_bf16((B, N, Hq, D), seed * 10 + 1)
    k = synth.normal_bf16((B, Hkv, S_max, D), seed * 10 + 2)
    v = synth.normal_bf16((B, Hkv, S_max, D), seed * 10 + 3)
    parents = np.stack([synth.draw_tree(N, 6, 4, rng) for _ in range(B)])
    mask, _, _ = oracle.tree_mask(parents)      # any valid mask serves; built on the CPU
    return dict(q=q, k=k, v=v, kv_len=np.asarray(kv_len, dtype=np.int32), mask=mask,
                qd=gu.bf16_dev(q), kd=gu.bf16_dev(k), vd=gu.bf16_dev(v), lend=gu.i32_dev(kv_len), maskd=gu.u64_dev(mask))


def _static(p, scale):
    from paper_2509_15235_b200 import binding
    B, N, Hq, D = p["q"].shape
    out = torch.full((B, N, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, Hq, N), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.tree_verify_attn_static(p["qd"], p["kd"], p["vd"], p["lend"], p["maskd"], scale, out, lse, status)
    torch.cuda.synchronize()
    return out.float().cpu().numpy(), lse.cpu().numpy(), int(status.item())


def test_static_entry_matches_regular_entry_on_two_calls_in_a_row():
    import gpu_util as gu
    p1 = _problem(1, 2, 60, 8, 8, 128, 1536, [1400, 901])       # several splits per head
    p2 = _problem(2, 1, 23, 14, 2, 128, 640, [555])             # different shape, GQA, shorter
    s1, s2 = 1 / math.sqrt(128), 0.07
    got1 = _static(p1, s1)
    got2 = _static(p2, s2)                                      # runs on top of p1's leftovers
    import oracle
    for p, s, got in ((p1, s1, got1), (p2, s2, got2)):
        want, want_lse, status = gu.run_attn(p["q"], p["k"], p["v"], p["kv_len"], p["mask"], s)
        assert status == 0 and got[2] == 0
        assert not np.isnan(got[0]).any()
        assert np.abs(got[0] - want).max() <= TOL
        assert np.abs(got[1] - want_lse).max() <= 2e-3
        # and against the oracle itself, not only against the other entry point
        ref, ref_lse = oracle.tree_attn(p["q"], p["k"], p["v"], p["kv_len"], p["mask"], s)
        assert np.abs(got[0] - ref).max() <= TOL
        assert np.abs(got[1] - ref_lse).max() <= 2e-3


def test_static_entry_rejects_problems_beyond_its_scratch_and_bad_arguments():
    from paper_2509_15235_b200 import binding
    # 8 sequences x 40 kv heads = 320 units of 64 rows: more than the 16 MiB array takes at D = 128
    B, N, H, D, S_max = 8, 60, 40, 128, 128
    q = torch.zeros((B, N, H, D), dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros((B, H, S_max, D), dtype=torch.bfloat16, device="cuda")
    lens = torch.zeros(B, dtype=torch.int32, device="cuda")
    mask = torch.ones((B, N, 1), dtype=torch.int64, device="cuda")
    with pytest.raises(binding.VispecError) as e:
        binding.tree_verify_attn_static(q, kv, kv, lens, mask, 1.0, torch.empty_like(q))
    assert e.value.code == -10
    with pytest.raises(binding.VispecError) as e:                # head dim outside {64, 128}
        binding.tree_verify_attn_static(q[:1, :, :2, :96].contiguous(), kv[:1, :2, :, :96].contiguous(),
                                        kv[:1, :2, :, :96].contiguous(), lens[:1], mask[:1], 1.0,
                                        torch.empty((1, N, 2, 96), dtype=torch.bfloat16, device="cuda"))
    assert e.value.code == -3


def test_static_entry_flags_an_overlong_sequence_in_the_callers_status_word():
    p = _problem(3, 2, 8, 4, 4, 64, 128, [125, 90])             # 125 + 8 > 128
    out, lse, status = _static(p, 0.125)
    assert status == -4 and (out[0] == 0).all()
    import oracle
    want, _ = oracle.tree_attn(p["q"][1:], p["k"][1:], p["v"][1:], [90], p["mask"][1:], 0.125)
    assert np.abs(out[1] - want[0]).max() <= TOL
