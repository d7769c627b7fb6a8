"""Seeded synthetic inputs for the draft-tree verification path.

This module only *draws* inputs (random K/V/Q tensors, random draft trees, random
token ids).  It contains none of the method's arithmetic: no mask construction, no
attention, no acceptance rule, no compaction.  Both the CUDA path's tests and the
CPU oracle's tests consume its buffers; it imports neither of them.

Workloads (paper, Sec. 5.1 names the target models LLaVA-v1.6-Vicuna-7B/13B and
Qwen2.5-VL-3B/7B; Sec. 5.3 says image embeddings number in the thousands; App. A
fixes the paper's own tree at 30 draft tokens, depth 3, top-8 expansion):

    tiny        B1,  4/4 heads,  D64,  S=256 (64 image + 192 text), 8-node tree
    llava7b     B1, 32/32 heads, D128, S=2880 image + 1024 text,   60-node tree, 32 layers
    qwen7b      B1, 28/4 heads,  D128, S=1296 image + 2048 text,   60-node tree, 28 layers
    llava13b_b4 B4, 40/40 heads, D128, S uniform in [3000,5000],    60-node trees, 40 layers
    qwen3b_*    16/2 heads, D128, S in {2k,8k,16k,32k}, N in {16,60,128}, B in {1,4,8}
    paper_tree  like llava7b but the paper's own tree: 31 nodes (root + 30), depth 3, branching 8

bf16 values are carried as numpy uint16 bit patterns (numpy has no bfloat16).
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional

import numpy as np

__all__ = [
    "VerifyConfig", "CONFIGS", "get_config", "f32_to_bf16_bits", "bf16_bits_to_f32",
    "normal_bf16", "draw_tree", "draw_ids", "draw_kv_len", "make_tree_inputs",
    "make_layer_tensors", "tensor_seed",
]


@dataclasses.dataclass(frozen=True)
class VerifyConfig:
    """Shape of one verification workload (one row of the configuration list)."""
    name: str
    config_id: int
    B: int            # sequences
    Hq: int           # query heads
    Hkv: int          # key/value heads
    D: int            # head dimension
    n_image: int      # image-token slots at the front of the cache
    S_lo: int         # committed length, inclusive lower bound
    S_hi: int         # committed length, inclusive upper bound (== S_lo: fixed length)
    N: int            # tree nodes including the root
    max_depth: int    # deepest node depth allowed (root has depth 0)
    max_children: int  # branching cap (0 = unlimited)
    layers: int
    vocab: int
    p_match: float

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def S_max(self) -> int:
        """Allocated slots per (sequence, kv head): longest prefix + tree, rounded up to 128."""
        need = self.S_hi + self.N
        return (need + 127) // 128 * 128

    def kv_bytes_per_layer(self, kv_len: np.ndarray) -> int:
        """Bytes of K and V rows the attention of one layer must read (bf16)."""
        return int(sum(2 * (int(s) + self.N) * self.Hkv * self.D * 2 for s in kv_len))


def _mk(name, cid, B, Hq, Hkv, D, n_img, S_lo, S_hi, N, depth, br, layers, vocab, p):
    return VerifyConfig(name, cid, B, Hq, Hkv, D, n_img, S_lo, S_hi, N, depth, br, layers, vocab, p)


CONFIGS: Dict[str, VerifyConfig] = {}


def _register(c: VerifyConfig) -> None:
    CONFIGS[c.name] = c


_register(_mk("tiny", 1, 1, 4, 4, 64, 64, 256, 256, 8, 3, 0, 1, 1000, 0.7))
_register(_mk("llava7b", 2, 1, 32, 32, 128, 2880, 3904, 3904, 60, 6, 4, 32, 32000, 0.7))
_register(_mk("qwen7b", 3, 1, 28, 4, 128, 1296, 3344, 3344, 60, 6, 4, 28, 152064, 0.6))
_register(_mk("llava13b_b4", 4, 4, 40, 40, 128, 2880, 3000, 5000, 60, 6, 4, 40, 32000, 0.7))
_cid = 500
for _S in (2048, 8192, 16384, 32768):
    for _N in (16, 60, 128):
        for _B in (1, 4, 8):
            _register(_mk(f"qwen3b_S{_S}_N{_N}_B{_B}", _cid, _B, 16, 2, 128, 1296, _S, _S, _N,
                          6, 4, 36, 151936, 0.6))
            _cid += 1
_register(_mk("paper_tree", 6, 1, 32, 32, 128, 2880, 3904, 3904, 31, 3, 8, 32, 32000, 0.7))


def get_config(name: str) -> VerifyConfig:
    return CONFIGS[name]


# --------------------------------------------------------------------------- bf16 helpers

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns, round to nearest even (NaN kept quiet)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    r = (u >> np.uint32(16)) & np.uint32(1)
    r += np.uint32(0x7FFF)
    r += u
    r >>= np.uint32(16)
    out = r.astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns -> float32 (exact)."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------- generators

def tensor_seed(config_id: int, layer: int, tensor_id: int) -> int:
    """One seed per (workload, layer, tensor): 0x5EC0DE00 + 1000*config + 10*layer + tensor."""
    return 0x5EC0DE00 + 1000 * int(config_id) + 10 * int(layer) + int(tensor_id)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.SFC64(int(seed)))


def normal_bf16(shape, seed: int) -> np.ndarray:
    """i.i.d. N(0,1) drawn in float32 and rounded to bf16 bit patterns."""
    n = int(np.prod(shape))
    g = _rng(seed)
    out = np.empty(n, dtype=np.uint16)
    step = 1 << 24
    for lo in range(0, n, step):
        hi = min(n, lo + step)
        out[lo:hi] = f32_to_bf16_bits(g.standard_normal(hi - lo, dtype=np.float32))
    return out.reshape(shape)


def draw_tree(N: int, max_depth: int, max_children: int, rng: np.random.Generator) -> np.ndarray:
    """Random draft tree as a parent array: node 0 is the root (parent -1); node i >= 1 takes a
    parent drawn uniformly from the earlier nodes that may still take a child (depth below the
    cap, fewer children than the branching cap; 0 = no branching cap)."""
    parents = np.full(N, -1, dtype=np.int32)
    depth = np.zeros(N, dtype=np.int64)
    kids = np.zeros(N, dtype=np.int64)
    for i in range(1, N):
        ok = [j for j in range(i)
              if depth[j] < max_depth and (max_children <= 0 or kids[j] < max_children)]
        if not ok:
            raise ValueError("tree caps leave no eligible parent")
        p = ok[int(rng.integers(0, len(ok)))]
        parents[i] = p
        depth[i] = depth[p] + 1
        kids[p] += 1
    return parents


def draw_ids(parents: np.ndarray, vocab: int, p_match: float, rng: np.random.Generator):
    """target_ids uniform over the vocabulary; each non-root draft token copies the target's
    prediction at its parent with probability p_match, else is a uniform *different* token."""
    N = parents.shape[0]
    target = rng.integers(0, vocab, size=N, dtype=np.int64).astype(np.int32)
    draft = np.zeros(N, dtype=np.int32)
    draft[0] = int(rng.integers(0, vocab))  # ignored by the method: the root is already committed
    for i in range(1, N):
        want = int(target[parents[i]])
        if rng.random() < p_match:
            draft[i] = want
        else:
            other = int(rng.integers(0, vocab - 1))
            draft[i] = other if other < want else other + 1
    return draft, target


def draw_kv_len(cfg: VerifyConfig, rng: np.random.Generator) -> np.ndarray:
    if cfg.S_lo == cfg.S_hi:
        return np.full(cfg.B, cfg.S_lo, dtype=np.int32)
    return rng.integers(cfg.S_lo, cfg.S_hi + 1, size=cfg.B, dtype=np.int64).astype(np.int32)


def make_tree_inputs(cfg: VerifyConfig, seed_offset: int = 0) -> Dict[str, np.ndarray]:
    """Per-cycle integer inputs: parents, draft_ids, target_ids [B,N] and kv_len [B]."""
    rng = _rng(tensor_seed(cfg.config_id, 0, 9) + 7919 * seed_offset)
    kv_len = draw_kv_len(cfg, rng)
    parents = np.stack([draw_tree(cfg.N, cfg.max_depth, cfg.max_children, rng) for _ in range(cfg.B)])
    ids = [draw_ids(parents[b], cfg.vocab, cfg.p_match, rng) for b in range(cfg.B)]
    draft = np.stack([d for d, _ in ids])
    target = np.stack([t for _, t in ids])
    return {"parents": parents, "draft_ids": draft, "target_ids": target, "kv_len": kv_len}


def softmax_rows_f32(logits: np.ndarray) -> np.ndarray:
    """Row-wise softmax in float32 (an input recipe: what a model's head would hand over)."""
    z = logits - logits.max(axis=-1, keepdims=True)
    e = np.exp(z, dtype=np.float32)
    return (e / e.sum(axis=-1, keepdims=True, dtype=np.float32)).astype(np.float32)


def make_sampled_inputs(parents: np.ndarray, V: int, seed: int, sharpness: float = 6.0,
                        disagreement: float = 0.3) -> Dict[str, np.ndarray]:
    """Inputs of the sampled (temperature > 0) acceptance for given trees [B,N]:
    p_target = softmax(sharpness * g), p_draft = softmax(sharpness * (g + disagreement * h)) with g, h i.i.d.
    N(0,1) per (node, token): a few tokens carry most of the mass, the two models mostly agree; each non-root
    node's token is drawn from its parent's draft row (i.i.d., so siblings may repeat); uniforms in [0,1)."""
    B, N = parents.shape
    rng = _rng(seed)
    p = np.empty((B, N, V), dtype=np.float32)
    ph = np.empty((B, N, V), dtype=np.float32)
    for b in range(B):
        g = rng.standard_normal((N, V), dtype=np.float32)
        p[b] = softmax_rows_f32(np.float32(sharpness) * g)
        g += np.float32(disagreement) * rng.standard_normal((N, V), dtype=np.float32)
        ph[b] = softmax_rows_f32(np.float32(sharpness) * g)
    ids = np.zeros((B, N), dtype=np.int32)
    for b in range(B):
        rows: Dict[int, np.ndarray] = {}
        for i in range(1, N):
            par = int(parents[b, i])
            if par not in rows:
                w = ph[b, par].astype(np.float64)
                rows[par] = w / w.sum()
            ids[b, i] = int(rng.choice(V, p=rows[par]))
    return {"p_target": p, "p_draft": ph, "draft_ids": ids,
            "u_accept": rng.random((B, N), dtype=np.float32), "u_bonus": rng.random(B, dtype=np.float32)}


def make_rerank_candidates(B: int, depth: int, width: int, vocab: int, seed: int) -> Dict[str, np.ndarray]:
    """Candidates of a level-by-level tree expansion (the input of the rerank): level 1 holds `width` children
    of the root, every later level `width` children of each of `width` candidates of the level before (drawn at
    random: which ones a draft model would expand is its business, not this generator's), so
    M = width + (depth - 1) * width^2 (136 for depth 3, width 8).  A child's score is its parent's plus the log
    of its share of a random split of the unit mass into width + 1 parts (cubed exponentials: a few children carry
    most of it, the last part stands for the rest of the vocabulary); tokens are distinct random ids."""
    rng = _rng(seed)
    M = width + (depth - 1) * width * width
    parent = np.full((B, M), -1, dtype=np.int32)
    token = np.zeros((B, M), dtype=np.int32)
    score = np.zeros((B, M), dtype=np.float32)

    def expand():
        w = rng.standard_exponential(width + 1) ** 3
        share = (w / w.sum())[:width]
        tok = rng.choice(vocab, size=width, replace=False)
        return tok.astype(np.int32), np.log(np.maximum(share, 1e-30)).astype(np.float32)

    for b in range(B):
        tok, lp = expand()
        token[b, :width], score[b, :width] = tok, lp
        level = list(range(width))
        n = width
        for _ in range(1, depth):
            best = [level[j] for j in rng.permutation(len(level))[:width]]
            level = []
            for par in sorted(best):
                tok, lp = expand()
                token[b, n:n + width] = tok
                score[b, n:n + width] = score[b, par] + lp
                parent[b, n:n + width] = par
                level.extend(range(n, n + width))
                n += width
    return {"cand_parent": parent, "cand_token": token, "cand_score": score}


def make_layer_tensors(cfg: VerifyConfig, layer: int, S_max: Optional[int] = None,
                       seed_offset: int = 0) -> Dict[str, np.ndarray]:
    """One layer's bf16 tensors as uint16 bit patterns:
    q [B,N,Hq,D]; k_cache, v_cache [B,Hkv,S_max,D] (every slot filled, so the tree rows at
    slots kv_len..kv_len+N-1 are present wherever kv_len falls)."""
    S_max = cfg.S_max if S_max is None else int(S_max)
    off = 100000 * seed_offset
    q = normal_bf16((cfg.B, cfg.N, cfg.Hq, cfg.D), tensor_seed(cfg.config_id, layer, 1) + off)
    k = normal_bf16((cfg.B, cfg.Hkv, S_max, cfg.D), tensor_seed(cfg.config_id, layer, 2) + off)
    v = normal_bf16((cfg.B, cfg.Hkv, S_max, cfg.D), tensor_seed(cfg.config_id, layer, 3) + off)
    return {"q": q, "k_cache": k, "v_cache": v}
