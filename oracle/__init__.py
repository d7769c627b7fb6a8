"""Python face of the CPU fp64 oracle (``vispec_oracle.c``).

TEST INFRASTRUCTURE ONLY.  The tests, the smoke check and the benchmark's CPU-baseline leg
call this; the product package never imports it, and this package never imports the product.
Every function cites the passage it follows in ``vispec_oracle.c``; nothing here is pinned to
itself: the pins live in the CPU tests (closed forms of Eq. 3 and Eq. 4, causal attention from a
library routine, hand-worked trees, brute force over every tree of at most 8 nodes).

bf16 tensors are numpy ``uint16`` bit patterns; outputs of the attention are ``float64``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "vispec_oracle.c")
_LIB = os.path.join(_HERE, "libvispec_oracle.so")
_lib: Optional[ctypes.CDLL] = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP, -O2).  Returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        for name in ("oracle_tree_mask", "oracle_tree_attn", "oracle_accept", "oracle_kv_compact",
                     "oracle_num_threads", "oracle_rope_rows", "oracle_accept_sampled", "oracle_tree_rerank"):
            getattr(_lib, name).restype = ctypes.c_int
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    """Threads the attention oracle runs on (OpenMP's maximum)."""
    return int(_load().oracle_num_threads())


def tree_mask(parents) -> Tuple[np.ndarray, np.ndarray, bool]:
    """parents [B,N] int32 -> (mask [B,N,W] uint64, depth [B,N] int32, all_parents_valid)."""
    parents = _c(parents, np.int32)
    B, N = parents.shape
    W = (N + 63) // 64
    mask = np.zeros((B, N, W), dtype=np.uint64)
    depth = np.zeros((B, N), dtype=np.int32)
    rc = _load().oracle_tree_mask(_p(parents), B, N, _p(mask), _p(depth))
    return mask, depth, rc == 0


def tree_attn(q, k_cache, v_cache, kv_len, mask, scale: float, want_lse: bool = True):
    """q [B,N,Hq,D], caches [B,Hkv,S_max,D] (uint16 bf16 bits), kv_len [B], mask [B,N,W] uint64
    -> (out [B,N,Hq,D] float64, lse [B,Hq,N] float64 or None)."""
    q = _c(q, np.uint16); k_cache = _c(k_cache, np.uint16); v_cache = _c(v_cache, np.uint16)
    kv_len = _c(kv_len, np.int32); mask = _c(mask, np.uint64)
    B, N, Hq, D = q.shape
    _, Hkv, S_max, _ = k_cache.shape
    assert v_cache.shape == k_cache.shape and mask.shape == (B, N, (N + 63) // 64)
    out = np.zeros((B, N, Hq, D), dtype=np.float64)
    lse = np.zeros((B, Hq, N), dtype=np.float64) if want_lse else None
    rc = _load().oracle_tree_attn(_p(q), _p(k_cache), _p(v_cache), _p(kv_len), _p(mask),
                                  B, N, Hq, Hkv, D, S_max, ctypes.c_double(scale), _p(out),
                                  _p(lse) if want_lse else None)
    if rc != 0:
        raise ValueError(f"oracle_tree_attn rejected its arguments (code {rc})")
    return out, lse


def accept(draft_ids, target_ids, parents):
    """-> (path [B,N] int32 padded with -1, accept_len [B] int32, bonus [B] int32)."""
    draft_ids = _c(draft_ids, np.int32); target_ids = _c(target_ids, np.int32)
    parents = _c(parents, np.int32)
    B, N = parents.shape
    path = np.zeros((B, N), dtype=np.int32)
    alen = np.zeros(B, dtype=np.int32)
    bonus = np.zeros(B, dtype=np.int32)
    rc = _load().oracle_accept(_p(draft_ids), _p(target_ids), _p(parents), B, N, _p(path), _p(alen),
                               _p(bonus))
    if rc != 0:
        raise ValueError(f"oracle_accept rejected its arguments (code {rc})")
    return path, alen, bonus


def accept_sampled(draft_ids, parents, p, p_hat, u_accept, u_bonus):
    """Sampled acceptance.  p, p_hat [B,N,V] float32; u_accept [B,N], u_bonus [B] float32 in [0,1).
    -> (path [B,N] int32 padded with -1, accept_len [B], bonus [B], number of invalid sequences)."""
    draft_ids = _c(draft_ids, np.int32); parents = _c(parents, np.int32)
    p = _c(p, np.float32); p_hat = _c(p_hat, np.float32)
    u_accept = _c(u_accept, np.float32); u_bonus = _c(u_bonus, np.float32)
    B, N, V = p.shape
    assert p_hat.shape == p.shape and parents.shape == (B, N) and draft_ids.shape == (B, N)
    assert u_accept.shape == (B, N) and u_bonus.shape == (B,)
    path = np.zeros((B, N), dtype=np.int32)
    alen = np.zeros(B, dtype=np.int32)
    bonus = np.zeros(B, dtype=np.int32)
    rc = _load().oracle_accept_sampled(_p(draft_ids), _p(parents), _p(p), _p(p_hat), _p(u_accept), _p(u_bonus),
                                       B, N, V, _p(path), _p(alen), _p(bonus))
    if rc < 0:
        raise MemoryError("oracle_accept_sampled")
    return path, alen, bonus, rc


def tree_rerank(cand_parent, cand_token, cand_score, K: int):
    """Candidates [B,M] -> (parents [B,K+1], draft_ids [B,K+1], selected [B,K], number of invalid sequences)."""
    cand_parent = _c(cand_parent, np.int32); cand_token = _c(cand_token, np.int32)
    cand_score = _c(cand_score, np.float32)
    B, M = cand_parent.shape
    assert cand_token.shape == (B, M) and cand_score.shape == (B, M)
    parents = np.zeros((B, K + 1), dtype=np.int32)
    ids = np.zeros((B, K + 1), dtype=np.int32)
    sel = np.zeros((B, K), dtype=np.int32)
    rc = _load().oracle_tree_rerank(_p(cand_parent), _p(cand_token), _p(cand_score), B, M, K, _p(parents), _p(ids),
                                    _p(sel))
    if rc < 0:
        raise ValueError(f"oracle_tree_rerank rejected its arguments (code {rc})")
    return parents, ids, sel, rc


def kv_compact(k_cache, v_cache, path, accept_len, kv_len):
    """Returns (k_cache', v_cache', kv_len') as new arrays; the inputs are not modified."""
    k = _c(k_cache, np.uint16).copy(); v = _c(v_cache, np.uint16).copy()
    path = _c(path, np.int32); accept_len = _c(accept_len, np.int32); kv_len = _c(kv_len, np.int32)
    B, Hkv, S_max, D = k.shape
    N = path.shape[1]
    out_len = np.zeros(B, dtype=np.int32)
    rc = _load().oracle_kv_compact(_p(k), _p(v), _p(path), _p(accept_len), _p(kv_len), _p(out_len),
                                   B, N, Hkv, D, S_max)
    if rc != 0:
        raise ValueError(f"oracle_kv_compact rejected its arguments (code {rc})")
    return k, v, out_len


def rope_rows(q, k_new, v_new, positions, kv_len, k_cache, v_cache, theta: float):
    """Rotary embedding of the tree's q / k rows and placement of the k / v rows at slots kv_len + i.
    Returns (q', k_cache', v_cache', skipped) as new arrays; the inputs are not modified."""
    q = _c(q, np.uint16).copy(); k_new = _c(k_new, np.uint16); v_new = _c(v_new, np.uint16)
    positions = _c(positions, np.int32); kv_len = _c(kv_len, np.int32)
    kc = _c(k_cache, np.uint16).copy(); vc = _c(v_cache, np.uint16).copy()
    B, N, Hq, D = q.shape
    _, Hkv, S_max, _ = kc.shape
    assert k_new.shape == (B, N, Hkv, D) and v_new.shape == k_new.shape and positions.shape == (B, N)
    rc = _load().oracle_rope_rows(_p(q), _p(k_new), _p(v_new), _p(positions), _p(kv_len), _p(kc), _p(vc),
                                  ctypes.c_double(theta), B, N, Hq, Hkv, D, S_max)
    return q, kc, vc, rc
