"""Thin ctypes binding of libvispec.so: argument marshalling only.

Every step of the verification path runs in the library's CUDA kernels; torch is used here for
device memory and streams.  There is no CPU fallback: if the shared object is missing or CUDA is
unavailable the import of the library (``load()``) raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libvispec.so")

VISPEC_OK = 0
STATUS_NAMES = {
    0: "VISPEC_OK", -1: "VISPEC_E_NULL", -2: "VISPEC_E_ALIGN", -3: "VISPEC_E_SHAPE", -4: "VISPEC_E_RANGE",
    -5: "VISPEC_E_UNSUPPORTED", -6: "VISPEC_E_CUDA", -7: "VISPEC_E_TIMEOUT", -8: "VISPEC_E_BAD_TREE",
    -9: "VISPEC_E_UNREGISTERED", -10: "VISPEC_E_WORKSPACE", -11: "VISPEC_E_POSITIONS",
}
EXPORTS = [
    "vispec_strerror", "vispec_ctx_create", "vispec_ctx_destroy", "vispec_workspace_bytes",
    "vispec_ctx_set_workspace", "vispec_cache_register", "vispec_tree_mask_build",
    "vispec_tree_verify_attn", "vispec_accept", "vispec_kv_compact", "vispec_status_poll",
    "vispec_launch_count", "vispec_tree_verify_attn_static", "vispec_ctx_set_option", "vispec_accept_commit", "vispec_stream_probe", "vispec_rope_tree_rows", "vispec_accept_sampled", "vispec_tree_rerank",
    "vispec_cache_register_paged", "vispec_tree_verify_attn_paged", "vispec_kv_compact_paged",
    "vispec_accept_commit_paged", "vispec_rope_tree_rows_paged", "vispec_selftest_bounded_wait",
    "vispec_rope_table_build", "vispec_rope_table_bytes", "vispec_tree_verify_attn_rope",
]
OPT_EARLY_PREFETCH = 1
OPT_FORCE_GENERIC = 2
OPT_SPLIT_FORM = 3
OPT_KV_LEN_HINT = 4
OPT_CHECK_POSITIONS = 5


class VispecShape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("B_max", "N_max", "Hq", "Hkv", "D", "S_max", "layers")]


class VispecError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {STATUS_NAMES.get(code, code)} ({strerror(code)})")


_lib: Optional[ctypes.CDLL] = None


def load() -> ctypes.CDLL:
    """dlopen the in-tree library.  Fails loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2509_15235_b200.build` "
                              "(there is no fallback path)")
        lib = ctypes.CDLL(LIB_PATH)
        vp, ci, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
        lib.vispec_strerror.restype = ctypes.c_char_p
        lib.vispec_strerror.argtypes = [ci]
        sigs = {
            "vispec_ctx_create": [ctypes.POINTER(vp), ctypes.POINTER(VispecShape), ci],
            "vispec_ctx_destroy": [vp],
            "vispec_workspace_bytes": [vp, ctypes.POINTER(ctypes.c_size_t)],
            "vispec_ctx_set_workspace": [vp, vp, ctypes.c_size_t],
            "vispec_cache_register": [vp, ci, vp, vp],
            "vispec_ctx_set_option": [vp, ci, ci],
            "vispec_tree_mask_build": [vp, vp, ci, ci, vp, vp, vp],
            "vispec_tree_verify_attn": [vp, ci, vp, vp, vp, vp, vp, vp, ci, ci, cf, vp, vp, vp],
            "vispec_accept": [vp, vp, vp, vp, ci, ci, vp, vp, vp, vp],
            "vispec_kv_compact": [vp, ci, ci, vp, vp, vp, vp, ci, ci, vp],
            "vispec_accept_commit": [vp, ci, ci, vp, vp, vp, vp, ci, ci, vp, vp, vp, vp, vp],
            "vispec_stream_probe": [vp, ci, vp, ci, ci, vp],
            "vispec_accept_sampled": [vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, vp, vp, vp, vp],
            "vispec_tree_rerank": [vp, vp, vp, vp, ci, ci, ci, vp, vp, vp, vp],
            "vispec_cache_register_paged": [vp, ci, vp, vp, ci, ci, ci],
            "vispec_tree_verify_attn_paged": [vp, ci, vp, vp, vp, ci, vp, ci, ci, cf, vp, vp, vp],
            "vispec_kv_compact_paged": [vp, ci, ci, vp, vp, vp, vp, ci, vp, ci, ci, vp],
            "vispec_accept_commit_paged": [vp, ci, ci, vp, vp, vp, vp, vp, ci, ci, ci, vp, vp, vp, vp, vp],
            "vispec_rope_tree_rows_paged": [vp, ci, vp, vp, vp, vp, vp, vp, ci, ci, ci, cf, vp],
            "vispec_rope_tree_rows": [vp, ci, vp, vp, vp, vp, vp, ci, ci, cf, vp],
            "vispec_status_poll": [vp, ctypes.POINTER(ci), vp],
            "vispec_launch_count": [vp, ctypes.POINTER(ctypes.c_uint64)],
            "vispec_selftest_bounded_wait": [vp, ctypes.c_longlong, vp],
            "vispec_rope_table_build": [vp, vp, ci, ci, cf, vp, vp],
            "vispec_rope_table_bytes": [vp, ci, ci, ctypes.POINTER(ctypes.c_size_t)],
            "vispec_tree_verify_attn_rope": [vp, ci, vp, vp, vp, vp, vp, vp, ci, ci, cf, vp, vp, vp],
            "vispec_tree_verify_attn_static": [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, vp, vp, vp, vp],
        }
        for name, argtypes in sigs.items():
            fn = getattr(lib, name)
            fn.restype = ci
            fn.argtypes = argtypes
        _lib = lib
    return _lib


def strerror(code: int) -> str:
    return load().vispec_strerror(int(code)).decode()


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device pointers must come from contiguous CUDA tensors"
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(code: int, where: str) -> None:
    if code != VISPEC_OK:
        raise VispecError(code, where)


def tree_verify_attn_static(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor,
                            kv_len: torch.Tensor, tree_mask: torch.Tensor, scale: float, out: torch.Tensor,
                            lse: Optional[torch.Tensor] = None, status_word: Optional[torch.Tensor] = None) -> None:
    """vispec_tree_verify_attn_static: the attention for callers that cannot allocate device memory
    (no context, no workspace; scratch is a fixed array inside the library).  One C call on torch's
    current stream; raises VispecError(VISPEC_E_WORKSPACE) when the problem exceeds the built-in scratch."""
    B, N, Hq, D = q.shape
    _, Hkv, S_max, _ = k_cache.shape
    _check(load().vispec_tree_verify_attn_static(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(kv_len),
                                                 _ptr(tree_mask), B, N, Hq, Hkv, D, S_max, ctypes.c_float(scale),
                                                 _ptr(out), _ptr(lse), _ptr(status_word), _stream()),
           "vispec_tree_verify_attn_static")


class VerifyContext:
    """Owns a ``vispec_ctx`` plus the torch-allocated workspace it points at.

    Method names mirror the C entry points; each is one C call on torch's current stream.
    """

    def __init__(self, B_max: int, N_max: int, Hq: int, Hkv: int, D: int, S_max: int, layers: int,
                 device: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("libvispec needs a CUDA device (no CPU fallback exists)")
        self.lib = load()
        self.shape = VispecShape(B_max, N_max, Hq, Hkv, D, S_max, layers)
        self.device = torch.device("cuda", device)
        h = ctypes.c_void_p()
        _check(self.lib.vispec_ctx_create(ctypes.byref(h), ctypes.byref(self.shape), device), "vispec_ctx_create")
        self.handle = h
        n = ctypes.c_size_t()
        _check(self.lib.vispec_workspace_bytes(self.handle, ctypes.byref(n)), "vispec_workspace_bytes")
        self.workspace = torch.empty(n.value, dtype=torch.uint8, device=self.device)
        _check(self.lib.vispec_ctx_set_workspace(self.handle, _ptr(self.workspace), n.value),
               "vispec_ctx_set_workspace")
        self._caches = {}

    def close(self) -> None:
        if getattr(self, "handle", None):
            self.lib.vispec_ctx_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def ctx_set_option(self, option: int, value: int) -> None:
        _check(self.lib.vispec_ctx_set_option(self.handle, option, value), "vispec_ctx_set_option")

    # -- registration ---------------------------------------------------------------------------
    def cache_register(self, layer: int, k_cache: torch.Tensor, v_cache: torch.Tensor) -> None:
        _check(self.lib.vispec_cache_register(self.handle, layer, _ptr(k_cache), _ptr(v_cache)),
               "vispec_cache_register")
        self._caches[layer] = (k_cache, v_cache)   # keep the tensors alive

    # -- hot calls --------------------------------------------------------------------------------
    def tree_mask_build(self, parents: torch.Tensor, tree_mask: torch.Tensor,
                        depth: Optional[torch.Tensor] = None) -> None:
        B, N = parents.shape
        _check(self.lib.vispec_tree_mask_build(self.handle, _ptr(parents), B, N, _ptr(tree_mask), _ptr(depth),
                                               _stream()), "vispec_tree_mask_build")

    def tree_verify_attn(self, layer: int, q: torch.Tensor, kv_len: torch.Tensor, tree_mask: torch.Tensor,
                         scale: float, out: torch.Tensor, lse: Optional[torch.Tensor] = None,
                         positions: Optional[torch.Tensor] = None, k_cache: Optional[torch.Tensor] = None,
                         v_cache: Optional[torch.Tensor] = None) -> None:
        B, N = q.shape[0], q.shape[1]
        _check(self.lib.vispec_tree_verify_attn(self.handle, layer, _ptr(q), _ptr(k_cache), _ptr(v_cache),
                                                _ptr(kv_len), _ptr(tree_mask), _ptr(positions), B, N,
                                                ctypes.c_float(scale), _ptr(out), _ptr(lse), _stream()),
               "vispec_tree_verify_attn")

    def accept(self, draft_ids: torch.Tensor, target_ids: torch.Tensor, parents: torch.Tensor,
               path: torch.Tensor, accept_len: torch.Tensor, bonus: torch.Tensor) -> None:
        B, N = parents.shape
        _check(self.lib.vispec_accept(self.handle, _ptr(draft_ids), _ptr(target_ids), _ptr(parents), B, N,
                                      _ptr(path), _ptr(accept_len), _ptr(bonus), _stream()), "vispec_accept")

    def kv_compact(self, layer_begin: int, layer_end: int, path: torch.Tensor, accept_len: torch.Tensor,
                   kv_len: torch.Tensor, kv_len_out: Optional[torch.Tensor] = None) -> None:
        B, N = path.shape
        _check(self.lib.vispec_kv_compact(self.handle, layer_begin, layer_end, _ptr(path), _ptr(accept_len),
                                          _ptr(kv_len), _ptr(kv_len_out), B, N, _stream()), "vispec_kv_compact")

    def accept_commit(self, layer_begin: int, layer_end: int, draft_ids: torch.Tensor, target_ids: torch.Tensor,
                      parents: torch.Tensor, kv_len: torch.Tensor, path: torch.Tensor, accept_len: torch.Tensor,
                      bonus: torch.Tensor, kv_len_out: Optional[torch.Tensor] = None) -> None:
        B, N = parents.shape
        _check(self.lib.vispec_accept_commit(self.handle, layer_begin, layer_end, _ptr(draft_ids), _ptr(target_ids),
                                             _ptr(parents), _ptr(kv_len), B, N, _ptr(path), _ptr(accept_len),
                                             _ptr(bonus), _ptr(kv_len_out), _stream()), "vispec_accept_commit")

    def accept_sampled(self, draft_ids: torch.Tensor, parents: torch.Tensor, p_target: torch.Tensor,
                       p_draft: torch.Tensor, u_accept: torch.Tensor, u_bonus: torch.Tensor, path: torch.Tensor,
                       accept_len: torch.Tensor, bonus: torch.Tensor) -> None:
        B, N, V = p_target.shape
        _check(self.lib.vispec_accept_sampled(self.handle, _ptr(draft_ids), _ptr(parents), _ptr(p_target), _ptr(p_draft),
                                              _ptr(u_accept), _ptr(u_bonus), B, N, V, _ptr(path), _ptr(accept_len),
                                              _ptr(bonus), _stream()), "vispec_accept_sampled")

    def tree_rerank(self, cand_parent: torch.Tensor, cand_token: torch.Tensor, cand_score: torch.Tensor, K: int,
                    parents: torch.Tensor, draft_ids: torch.Tensor, selected: Optional[torch.Tensor]) -> None:
        B, M = cand_parent.shape
        _check(self.lib.vispec_tree_rerank(self.handle, _ptr(cand_parent), _ptr(cand_token), _ptr(cand_score), B, M, K,
                                           _ptr(parents), _ptr(draft_ids), _ptr(selected), _stream()),
               "vispec_tree_rerank")

    def cache_register_paged(self, layer: int, k_pool: torch.Tensor, v_pool: torch.Tensor,
                             token_major: bool = False) -> None:
        """Pools [num_blocks, Hkv, page_rows, D], or [num_blocks, page_rows, Hkv, D] with token_major."""
        num_blocks, page_rows = k_pool.shape[0], k_pool.shape[1 if token_major else 2]
        _check(self.lib.vispec_cache_register_paged(self.handle, layer, _ptr(k_pool), _ptr(v_pool), num_blocks, page_rows,
                                                    int(token_major)), "vispec_cache_register_paged")
        self._caches[layer] = (k_pool, v_pool)   # keep the tensors alive

    def tree_verify_attn_paged(self, layer: int, q: torch.Tensor, kv_len: torch.Tensor, block_table: torch.Tensor,
                               tree_mask: torch.Tensor, scale: float, out: torch.Tensor,
                               lse: Optional[torch.Tensor] = None) -> None:
        B, N = q.shape[0], q.shape[1]
        _check(self.lib.vispec_tree_verify_attn_paged(self.handle, layer, _ptr(q), _ptr(kv_len), _ptr(block_table),
                                                      block_table.shape[1], _ptr(tree_mask), B, N, ctypes.c_float(scale),
                                                      _ptr(out), _ptr(lse), _stream()), "vispec_tree_verify_attn_paged")

    def kv_compact_paged(self, layer_begin: int, layer_end: int, path: torch.Tensor, accept_len: torch.Tensor,
                         kv_len: torch.Tensor, block_table: torch.Tensor, kv_len_out: Optional[torch.Tensor]) -> None:
        B, N = path.shape
        _check(self.lib.vispec_kv_compact_paged(self.handle, layer_begin, layer_end, _ptr(path), _ptr(accept_len),
                                                _ptr(kv_len), _ptr(block_table), block_table.shape[1], _ptr(kv_len_out),
                                                B, N, _stream()), "vispec_kv_compact_paged")

    def accept_commit_paged(self, layer_begin: int, layer_end: int, draft_ids: torch.Tensor, target_ids: torch.Tensor,
                            parents: torch.Tensor, kv_len: torch.Tensor, block_table: torch.Tensor, path: torch.Tensor,
                            accept_len: torch.Tensor, bonus: torch.Tensor, kv_len_out: Optional[torch.Tensor]) -> None:
        B, N = parents.shape
        _check(self.lib.vispec_accept_commit_paged(self.handle, layer_begin, layer_end, _ptr(draft_ids), _ptr(target_ids),
                                                   _ptr(parents), _ptr(kv_len), _ptr(block_table), block_table.shape[1],
                                                   B, N, _ptr(path), _ptr(accept_len), _ptr(bonus), _ptr(kv_len_out),
                                                   _stream()), "vispec_accept_commit_paged")

    def rope_tree_rows_paged(self, layer: int, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                             positions: torch.Tensor, kv_len: torch.Tensor, block_table: torch.Tensor,
                             theta: float) -> None:
        B, N = positions.shape
        _check(self.lib.vispec_rope_tree_rows_paged(self.handle, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(positions),
                                                    _ptr(kv_len), _ptr(block_table), block_table.shape[1], B, N,
                                                    ctypes.c_float(theta), _stream()), "vispec_rope_tree_rows_paged")

    def rope_tree_rows(self, layer: int, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                       positions: torch.Tensor, kv_len: torch.Tensor, theta: float) -> None:
        B, N = positions.shape
        _check(self.lib.vispec_rope_tree_rows(self.handle, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(positions),
                                              _ptr(kv_len), B, N, ctypes.c_float(theta), _stream()),
               "vispec_rope_tree_rows")

    def rope_table_build(self, positions: torch.Tensor, theta: float, table: Optional[torch.Tensor] = None) -> torch.Tensor:
        """vispec_rope_table_build; allocates the table (a uint8 tensor of vispec_rope_table_bytes) unless one is given."""
        B, N = positions.shape
        if table is None:
            n = ctypes.c_size_t()
            _check(self.lib.vispec_rope_table_bytes(self.handle, B, N, ctypes.byref(n)), "vispec_rope_table_bytes")
            table = torch.empty(max(n.value, 16), dtype=torch.uint8, device=self.device)
        _check(self.lib.vispec_rope_table_build(self.handle, _ptr(positions), B, N, ctypes.c_float(theta), _ptr(table),
                                                _stream()), "vispec_rope_table_build")
        return table

    def tree_verify_attn_rope(self, layer: int, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                              rope_table: torch.Tensor, kv_len: torch.Tensor, tree_mask: torch.Tensor, scale: float,
                              out: torch.Tensor, lse: Optional[torch.Tensor] = None) -> None:
        B, N = q.shape[0], q.shape[1]
        _check(self.lib.vispec_tree_verify_attn_rope(self.handle, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(rope_table),
                                                     _ptr(kv_len), _ptr(tree_mask), B, N, ctypes.c_float(scale), _ptr(out),
                                                     _ptr(lse), _stream()), "vispec_tree_verify_attn_rope")

    def stream_probe(self, layer: int, kv_len: torch.Tensor, N: int) -> None:
        _check(self.lib.vispec_stream_probe(self.handle, layer, _ptr(kv_len), kv_len.shape[0], N, _stream()),
               "vispec_stream_probe")

    # -- diagnostics ------------------------------------------------------------------------------
    def status_poll(self) -> int:
        code = ctypes.c_int()
        _check(self.lib.vispec_status_poll(self.handle, ctypes.byref(code), _stream()), "vispec_status_poll")
        return code.value

    def selftest_bounded_wait(self, limit_cycles: int) -> None:
        _check(self.lib.vispec_selftest_bounded_wait(self.handle, limit_cycles, _stream()), "vispec_selftest_bounded_wait")

    def launch_count(self) -> int:
        n = ctypes.c_uint64()
        _check(self.lib.vispec_launch_count(self.handle, ctypes.byref(n)), "vispec_launch_count")
        return n.value
