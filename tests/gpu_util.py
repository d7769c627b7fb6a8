"""Helpers shared by the GPU parity tests: numpy <-> torch marshalling and a one-shot runner that
pushes one layer's seeded inputs through the C ABI."""
from __future__ import annotations

import numpy as np
import torch

from paper_2509_15235_b200 import binding


def bf16_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> CUDA bfloat16 tensor of the same shape."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def i32_dev(a) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


def u64_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint64).view(np.int64)).cuda()


def u64_host(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy().view(np.uint64)


def run_attn(q, k, v, kv_len, mask, scale, want_lse=True, B_max=None, N_max=None, split_form=0, early_prefetch=None):
    """One attention call through the C ABI.  Inputs are numpy (bf16 bits / int32 / uint64).
    Returns (out float32 [B,N,Hq,D], lse float32 [B,Hq,N] or None, status word)."""
    B, N, Hq, D = q.shape
    _, Hkv, S_max, _ = k.shape
    ctx = binding.VerifyContext(B_max or max(B, 1), N_max or N, Hq, Hkv, D, S_max, 1)
    if split_form:
        ctx.ctx_set_option(binding.OPT_SPLIT_FORM, split_form)
    if early_prefetch is not None:
        ctx.ctx_set_option(binding.OPT_EARLY_PREFETCH, int(early_prefetch))
    kd, vd = bf16_dev(k), bf16_dev(v)
    ctx.cache_register(0, kd, vd)
    qd = bf16_dev(q)
    out = torch.full((B, N, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, Hq, N), float("nan"), dtype=torch.float32, device="cuda") if want_lse else None
    ctx.tree_verify_attn(0, qd, i32_dev(kv_len), u64_dev(mask), scale, out, lse)
    torch.cuda.synchronize()
    status = ctx.status_poll()
    res = out.float().cpu().numpy(), (lse.cpu().numpy() if want_lse else None), status
    ctx.close()
    return res
