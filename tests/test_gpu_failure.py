"""Failure detection on the GPU without a fault: a bounded device-side wait that runs out, the status word it leaves,
the recovery of the context; the debug check of `positions`; the host hint for the expected cache length."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2509_15235_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 2e-2


def _inputs(B, N, Hq, Hkv, D, S_max, kv_len, seed):
    rng = np.random.Generator(np.random.Philox(seed))
    q = synth.normal_bf16((B, N, Hq, D), seed + 1)
    k = synth.normal_bf16((B, Hkv, S_max, D), seed + 2)
    v = synth.normal_bf16((B, Hkv, S_max, D), seed + 3)
    parents = np.stack([synth.draw_tree(N, 6, 4, rng) for _ in range(B)])
    mask, depth, _ = oracle.tree_mask(parents)
    return q, k, v, np.asarray(kv_len, dtype=np.int32), parents, mask, depth


def test_a_wait_that_runs_out_reports_timeout_and_the_context_recovers():
    """vispec_selftest_bounded_wait polls a barrier nobody arrives on: the kernel must come back, the status word must
    read VISPEC_E_TIMEOUT, the poll must clear the arrival counter the give-up left behind, and an attention call on
    the same context afterwards must be as good as one before."""
    from paper_2509_15235_b200 import binding
    import gpu_util as gu
    B, N, Hq, Hkv, D, S_max = 2, 24, 4, 4, 128, 1024
    q, k, v, kv_len, _, mask, _ = _inputs(B, N, Hq, Hkv, D, S_max, [900, 411], 40)
    scale = 1 / math.sqrt(D)
    want, _ = oracle.tree_attn(q, k, v, kv_len, mask, scale)
    ctx = binding.VerifyContext(B, N, Hq, Hkv, D, S_max, 1)
    ctx.ctx_set_option(binding.OPT_SPLIT_FORM, 1)            # the form that counts arrivals in the workspace
    kd, vd, qd = gu.bf16_dev(k), gu.bf16_dev(v), gu.bf16_dev(q)
    ctx.cache_register(0, kd, vd)
    kvd, md = gu.i32_dev(kv_len), gu.u64_dev(mask)

    def attend():
        out = torch.full((B, N, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        ctx.tree_verify_attn(0, qd, kvd, md, scale, out)
        torch.cuda.synchronize()
        return out.float().cpu().numpy()

    assert np.abs(attend() - want).max() <= TOL and ctx.status_poll() == 0
    counters = ctx.workspace[:64 * 1024].view(torch.int32)
    assert int(counters.abs().sum()) == 0
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    ctx.selftest_bounded_wait(400_000)                        # about 0.2 ms at 1.9 GHz
    t1.record()
    torch.cuda.synchronize()                                 # it returns: nothing hangs
    assert t0.elapsed_time(t1) < 100.0                       # the second waiter was released by the flag, not by its own 0.8 s
    assert int(counters[0]) == 1                             # what the give-up left behind
    assert ctx.status_poll() == -7                           # VISPEC_E_TIMEOUT, and the poll zeroes the counters
    torch.cuda.synchronize()
    assert int(counters.abs().sum()) == 0
    assert ctx.status_poll() == 0
    assert np.abs(attend() - want).max() <= TOL and ctx.status_poll() == 0
    with pytest.raises(binding.VispecError) as e:
        ctx.selftest_bounded_wait(0)
    assert e.value.code == -4
    ctx.close()


def test_positions_are_checked_on_request_and_the_accepted_path_keeps_them_contiguous():
    """positions = kv_len + depth: with VISPEC_OPT_CHECK_POSITIONS the attention call verifies it on the device (status
    word, nothing else changes).  And for the accepted path: positions[path[k]] == kv_len + k, the slot the commit
    moves that node's row to."""
    from paper_2509_15235_b200 import binding
    import gpu_util as gu
    B, N, Hq, Hkv, D, S_max = 3, 31, 4, 2, 128, 640
    q, k, v, kv_len, parents, mask, depth = _inputs(B, N, Hq, Hkv, D, S_max, [500, 0, 77], 50)
    scale = 1 / math.sqrt(D)
    ctx = binding.VerifyContext(B, N, Hq, Hkv, D, S_max, 1)
    kd, vd, qd = gu.bf16_dev(k), gu.bf16_dev(v), gu.bf16_dev(q)
    ctx.cache_register(0, kd, vd)
    kvd, pd = gu.i32_dev(kv_len), gu.i32_dev(parents)
    md = torch.zeros((B, N, 1), dtype=torch.int64, device="cuda")
    dd = torch.zeros((B, N), dtype=torch.int32, device="cuda")
    ctx.tree_mask_build(pd, md, dd)
    positions = (kvd[:, None] + dd).to(torch.int32).contiguous()
    assert np.array_equal(positions.cpu().numpy(), kv_len[:, None] + depth)
    outs = []
    for check, pos, want_status in ((0, positions, 0), (1, positions, 0), (1, positions + (torch.arange(N, device="cuda") == 5), -11),
                                    (0, positions + 3, 0)):
        ctx.ctx_set_option(binding.OPT_CHECK_POSITIONS, check)
        out = torch.full((B, N, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        ctx.tree_verify_attn(0, qd, kvd, md, scale, out, positions=pos.to(torch.int32).contiguous())
        torch.cuda.synchronize()
        assert ctx.status_poll() == want_status
        outs.append(out.float().cpu().numpy())
    want, _ = oracle.tree_attn(q, k, v, kv_len, mask, scale)
    for o in outs:
        assert np.abs(o - want).max() <= TOL
        assert np.array_equal(o, outs[0])                     # the check changes nothing of the result
    # accepted path: positions run kv_len, kv_len + 1, ... along it
    rng = np.random.Generator(np.random.Philox(51))
    target = rng.integers(0, 9, size=(B, N)).astype(np.int32)
    draft = np.where(rng.random((B, N)) < 0.8, np.take_along_axis(target, np.maximum(parents, 0), 1), 99).astype(np.int32)
    path = torch.zeros((B, N), dtype=torch.int32, device="cuda")
    alen = torch.zeros(B, dtype=torch.int32, device="cuda"); bonus = torch.zeros_like(alen)
    ctx.accept(gu.i32_dev(draft), gu.i32_dev(target), pd, path, alen, bonus)
    torch.cuda.synchronize()
    path, alen, pos = path.cpu().numpy(), alen.cpu().numpy(), positions.cpu().numpy()
    assert alen.max() >= 2
    for b in range(B):
        for kk in range(alen[b]):
            assert pos[b, path[b, kk]] == kv_len[b] + kk
    ctx.close()


@pytest.mark.parametrize("hint", [0, 2048])
def test_a_large_context_serving_short_sequences(hint):
    """Capacity 32 k slots, sequences of about 2 k tokens: the host's choice of form looks at the capacity unless it is
    given VISPEC_OPT_KV_LEN_HINT; either way the result is the oracle's (every output of one kv head's group)."""
    from paper_2509_15235_b200 import binding
    import gpu_util as gu
    B, N, Hq, Hkv, D, S_max = 2, 16, 16, 2, 128, 32768
    q, k, v, kv_len, _, mask, _ = _inputs(B, N, Hq, Hkv, D, S_max, [2048, 1777], 60)
    scale = 1 / math.sqrt(D)
    ctx = binding.VerifyContext(B, N, Hq, Hkv, D, S_max, 1)
    ctx.ctx_set_option(binding.OPT_KV_LEN_HINT, hint)
    ctx.cache_register(0, gu.bf16_dev(k), gu.bf16_dev(v))
    out = torch.full((B, N, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, Hq, N), float("nan"), dtype=torch.float32, device="cuda")
    ctx.tree_verify_attn(0, gu.bf16_dev(q), gu.i32_dev(kv_len), gu.u64_dev(mask), scale, out, lse)
    torch.cuda.synchronize()
    assert ctx.status_poll() == 0
    short = max(int(kv_len.max()) + N, 64)
    want, want_lse = oracle.tree_attn(q, k[:, :, :short], v[:, :, :short], kv_len, mask, scale)
    assert np.abs(out.float().cpu().numpy() - want).max() <= TOL
    assert np.abs(lse.cpu().numpy() - want_lse).max() <= 2e-3
    with pytest.raises(binding.VispecError):
        ctx.ctx_set_option(binding.OPT_KV_LEN_HINT, -1)
    ctx.close()
