"""Seeded synthetic inputs for the verify step (shapes, dtypes and value recipes only).

This module holds no arithmetic of the method itself: it draws random tensors, rounds them to
bf16 storage, and mixes probability vectors that the caller supplies.  It imports neither the
CUDA binding nor the CPU oracle, so both can be fed bit-identical arrays from here.

bf16 tensors are carried as ``numpy.uint16`` bit patterns (numpy has no bf16 type).

Notation (speculative sampling, Sec. 3; verification, Sec. 4.2): B sequences, S = 2B
classifier-free-guidance streams (conditional streams first, unconditional next), K drafted
tokens per sequence, H heads of dimension D, prefix KV length L, vocabulary V with valid ids
[v_begin, v_end).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np


@dataclass(frozen=True)
class VerifyConfig:
    name: str
    B: int            # sequences
    K: int            # drafted tokens per sequence
    H: int            # query heads
    H_kv: int         # key/value heads
    D: int            # head dimension
    L: int            # prefix KV length (the block's own K rows come on top)
    V: int            # output vocabulary (logit row length)
    v_begin: int      # first valid token id
    v_end: int        # one past the last valid token id
    cfg_scale: float
    temperature: float
    top_k: int        # <= 0: no filter
    q_recipe: str     # "own" | "mix" | "mix_row_uniform" | "disjoint"
    q_alpha: float = 0.7

    @property
    def S(self) -> int:
        return 2 * self.B

    @property
    def hidden(self) -> int:
        return self.H * self.D

    @property
    def M(self) -> int:           # token rows through the output head
        return self.S * self.K

    @property
    def L_cap(self) -> int:       # cache capacity per (stream, head)
        return self.L + self.K

    @property
    def V_valid(self) -> int:
        return self.v_end - self.v_begin


# The five workload shapes.  Generation settings of the paper (Sec. 5, "Model and Benchmark"):
# top-k 2000, temperature 1.0, guidance scale 3.0, 48x48 token grid.
CONFIGS: Dict[int, VerifyConfig] = {
    1: VerifyConfig("tiny", B=1, K=4, H=16, H_kv=16, D=64, L=128, V=16384, v_begin=0, v_end=16384,
                    cfg_scale=4.0, temperature=1.0, top_k=1000, q_recipe="own"),
    2: VerifyConfig("xl", B=8, K=5, H=20, H_kv=20, D=64, L=1144, V=16384, v_begin=0, v_end=16384,
                    cfg_scale=7.5, temperature=1.0, top_k=2000, q_recipe="mix", q_alpha=0.7),
    3: VerifyConfig("xxl", B=32, K=6, H=24, H_kv=24, D=64, L=1144, V=16384, v_begin=0, v_end=16384,
                    cfg_scale=7.5, temperature=1.0, top_k=2000, q_recipe="mix_row_uniform"),
    4: VerifyConfig("7b", B=4, K=6, H=32, H_kv=32, D=128, L=2400, V=65536, v_begin=4, v_end=8196,
                    cfg_scale=3.0, temperature=1.0, top_k=2000, q_recipe="mix", q_alpha=0.7),
    5: VerifyConfig("stress", B=64, K=8, H=20, H_kv=20, D=64, L=1024, V=16384, v_begin=0, v_end=16384,
                    cfg_scale=7.5, temperature=1.0, top_k=0, q_recipe="mix", q_alpha=0.5),
}
XL_PREFIX_SWEEP = (120, 376, 632, 888, 1144)
STRESS_ALPHAS = (0.0, 0.5, 0.9, 1.0)


def config(config_id: int, **overrides) -> VerifyConfig:
    cfg = CONFIGS[config_id]
    return replace(cfg, **overrides) if overrides else cfg


def seed_for(config_id: int, subcase: int = 0) -> int:
    return 1000 * config_id + subcase


# ------------------------------------------------------------------------------------------
# bf16 storage helpers (round-to-nearest-even on the fp32 bit pattern)
# ------------------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    bits = x.view(np.uint32).astype(np.uint64)
    rounded = bits + 0x7FFF + ((bits >> 16) & 1)
    return (rounded >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def _normal_bf16(rng: np.random.Generator, shape, std: float = 1.0) -> np.ndarray:
    return f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32) * np.float32(std))


# ------------------------------------------------------------------------------------------
# per-stage inputs
# ------------------------------------------------------------------------------------------
def make_attn_inputs(cfg: VerifyConfig, seed: int, ragged: bool = False) -> dict:
    """Q, K/V caches (block rows already in place) and prefix lengths; all values ~N(0,1) in bf16.

    ragged=True draws each stream's prefix length from [max(0, L - L//4), L].
    Cache slots past prefix_len + K are filled with N(0,1) too: the kernels must not read them
    into the result.
    """
    rng = np.random.default_rng(seed)
    S, K, H, Hkv, D, Lc = cfg.S, cfg.K, cfg.H, cfg.H_kv, cfg.D, cfg.L_cap
    q = _normal_bf16(rng, (S, K, H, D))
    k_cache = _normal_bf16(rng, (S, Hkv, Lc, D))
    v_cache = _normal_bf16(rng, (S, Hkv, Lc, D))
    if ragged:
        lo = max(0, cfg.L - cfg.L // 4)
        prefix_len = rng.integers(lo, cfg.L + 1, size=S).astype(np.int32)
    else:
        prefix_len = np.full(S, cfg.L, dtype=np.int32)
    return dict(q=q, k_cache=k_cache, v_cache=v_cache, prefix_len=prefix_len,
                sm_scale=np.float32(1.0 / np.sqrt(np.float32(D))))


def make_head_inputs(cfg: VerifyConfig, seed: int) -> dict:
    """Hidden states X ~N(0,1) and head weight W ~N(0,0.02), both bf16."""
    rng = np.random.default_rng(seed + 1)
    x = _normal_bf16(rng, (cfg.M, cfg.hidden), 1.0)
    w = _normal_bf16(rng, (cfg.V, cfg.hidden), 0.02)
    return dict(x=x, w=w)


def make_logits(cfg: VerifyConfig, seed: int, has_bonus_row: bool = False) -> np.ndarray:
    """fp32 logits [S, K(+1), V] with the spread the head would give: std 0.02*sqrt(hidden).

    Ids outside [v_begin, v_end) hold NaN so that any read of them shows up in the result.
    """
    rng = np.random.default_rng(seed + 2)
    rows = cfg.K + (1 if has_bonus_row else 0)
    std = np.float32(0.02 * np.sqrt(cfg.hidden))
    logits = rng.standard_normal((cfg.S, rows, cfg.V), dtype=np.float32) * std
    if cfg.v_begin > 0:
        logits[..., : cfg.v_begin] = np.nan
    if cfg.v_end < cfg.V:
        logits[..., cfg.v_end:] = np.nan
    return logits


def mask_odd_ids(logits: np.ndarray, cfg: VerifyConfig) -> np.ndarray:
    """Disjoint-support case: odd token ids get -inf in every stream (target lives on even ids)."""
    out = logits.copy()
    ids = np.arange(cfg.V)
    odd = (ids % 2 == 1) & (ids >= cfg.v_begin) & (ids < cfg.v_end)
    out[..., odd] = -np.inf
    return out


def random_probs(cfg: VerifyConfig, seed: int, only_odd: bool = False) -> np.ndarray:
    """r[B, K, V]: a random dense distribution over the valid ids (normalised exp of N(0,1) draws)."""
    rng = np.random.default_rng(seed + 3)
    z = rng.standard_normal((cfg.B, cfg.K, cfg.V))
    ids = np.arange(cfg.V)
    valid = (ids >= cfg.v_begin) & (ids < cfg.v_end)
    if only_odd:
        valid &= ids % 2 == 1
    z = np.where(valid, z, -np.inf)
    e = np.exp(z - z.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def mix_q(p: Optional[np.ndarray], r: np.ndarray, alpha) -> np.ndarray:
    """q = alpha * p + (1 - alpha) * r as fp32; p is whatever target probabilities the caller passes."""
    alpha = np.asarray(alpha, dtype=np.float64)
    if p is None:
        return r.astype(np.float32)
    while alpha.ndim and alpha.ndim < r.ndim:
        alpha = alpha[..., None]
    return (alpha * np.asarray(p, dtype=np.float64) + (1.0 - alpha) * r).astype(np.float32)


def row_alphas(cfg: VerifyConfig, seed: int, lo: float = 0.3, hi: float = 0.95) -> np.ndarray:
    rng = np.random.default_rng(seed + 4)
    return rng.uniform(lo, hi, size=(cfg.B, cfg.K))


def draw_drafts(q: np.ndarray, seed: int) -> np.ndarray:
    """draft[b, i] ~ q[b, i, :] by inverse CDF with its own uniforms."""
    rng = np.random.default_rng(seed + 5)
    B, K, V = q.shape
    u = rng.random((B, K))
    cdf = np.cumsum(q.astype(np.float64), axis=-1)
    t = u * cdf[..., -1]
    idx = (cdf > t[..., None]).argmax(axis=-1)
    return idx.astype(np.int32)


def draw_uniforms(cfg: VerifyConfig, seed: int) -> dict:
    """u_accept[B, K] and u_resample[B, K+1], fp32 in [0, 1)."""
    rng = np.random.default_rng(seed + 6)
    u_acc = rng.random((cfg.B, cfg.K), dtype=np.float32)
    u_res = rng.random((cfg.B, cfg.K + 1), dtype=np.float32)
    # float32 rounding of values just below 1 can give exactly 1.0; keep the interval half-open
    one_below = np.nextafter(np.float32(1.0), np.float32(0.0))
    return dict(u_accept=np.minimum(u_acc, one_below), u_resample=np.minimum(u_res, one_below))


def make_q(cfg: VerifyConfig, seed: int, p: Optional[np.ndarray]) -> np.ndarray:
    """Draft distribution per the config's recipe; p = target probabilities [B, K, V] where needed."""
    if cfg.q_recipe == "own":
        return mix_q(None, random_probs(cfg, seed), 0.0)
    if cfg.q_recipe == "disjoint":
        return mix_q(None, random_probs(cfg, seed, only_odd=True), 0.0)
    if p is None:
        raise ValueError(f"q recipe {cfg.q_recipe!r} needs target probabilities")
    r = random_probs(cfg, seed)
    if cfg.q_recipe == "mix":
        return mix_q(p, r, cfg.q_alpha)
    if cfg.q_recipe == "mix_row_uniform":
        return mix_q(p, r, row_alphas(cfg, seed))
    raise ValueError(cfg.q_recipe)


# ------------------------------------------------------------------------------------------
# candidate trees (several candidates per depth, Sec. 4.2): topology and draws only
# ------------------------------------------------------------------------------------------
def make_tree(branching=(3, 2, 2)) -> dict:
    """Full tree in breadth-first order with `branching[d]` children under every node of depth d.

    Returns child_begin [N+1], node_depth [N], node_slot [N] (which of its parent's candidates a node
    is) and node_q [N]: candidate `slot` of depth d draws from draft row d * max(branching) + slot,
    i.e. every candidate of a level comes from its own draft head.
    """
    width = max(branching)
    depth, slot, level = [0], [0], [0]
    child_begin = []
    n = 1
    for d, c in enumerate(branching):
        nxt = []
        for _ in level:
            child_begin.append(n)
            for j in range(c):
                depth.append(d + 1); slot.append(j); nxt.append(n); n += 1
        level = nxt
    child_begin += [n] * (len(level) + 1)
    depth = np.array(depth, np.int32); slot = np.array(slot, np.int32)
    node_q = np.where(depth > 0, (depth - 1) * width + slot, 0).astype(np.int32)
    return dict(child_begin=np.array(child_begin, np.int32), node_depth=depth, node_slot=slot, node_q=node_q,
                N=n, NQ=len(branching) * width)


def tree_ancestor_masks(child_begin: np.ndarray) -> np.ndarray:
    """anc_mask[i] (uint64): bit m set iff node m lies on the path from the root to node i, i included.
    Index bookkeeping for the attention mask of a tree with at most 64 nodes."""
    N = len(child_begin) - 1
    if N > 64:
        raise ValueError("a mask word holds 64 nodes")
    parent = np.full(N, -1, np.int64)
    for n in range(N):
        parent[child_begin[n]:child_begin[n + 1]] = n
    masks = np.zeros(N, np.uint64)
    for i in range(N):
        m, n = 0, i
        while n >= 0:
            m |= 1 << int(n)
            n = parent[n]
        masks[i] = np.uint64(m)
    return masks


def chain_masks(K: int) -> np.ndarray:
    """The masks of a plain chain of K drafts: position i sees block rows 0..i."""
    return np.array([(1 << (i + 1)) - 1 for i in range(K)], dtype=np.uint64)


def draw_tree_tokens(q: np.ndarray, tree: dict, seed: int) -> np.ndarray:
    """node_token[B, N]: one draw per (sequence, depth, candidate slot) from its draft row, shared by all
    nodes of that depth and slot (the tree is the Cartesian product of the per-position samples)."""
    rng = np.random.default_rng(seed + 7)
    B, NQ, V = q.shape
    u = rng.random((B, NQ))
    cdf = np.cumsum(q.astype(np.float64), axis=-1)
    draw = (cdf > (u * cdf[..., -1])[..., None]).argmax(axis=-1).astype(np.int32)     # [B, NQ]
    tok = draw[:, tree["node_q"]]
    tok[:, 0] = 0
    return np.ascontiguousarray(tok)


def draw_tree_uniforms(B: int, N: int, seed: int) -> dict:
    rng = np.random.default_rng(seed + 8)
    one_below = np.nextafter(np.float32(1.0), np.float32(0.0))
    return dict(u_accept=np.minimum(rng.random((B, N), dtype=np.float32), one_below),
                u_resample=np.minimum(rng.random((B, N), dtype=np.float32), one_below))


# ------------------------------------------------------------------------------------------
# draft-head outputs for the speculation cache and the sampling pool (Sec. 4.2): random rows only
# ------------------------------------------------------------------------------------------
def make_head_probs(B: int, R: int, V: int, v_begin: int, v_end: int, seed: int, sharp: float = 4.0) -> np.ndarray:
    """[B, R, V] fp32 distributions over the valid ids, normalised exp of sharp * N(0,1): a few ids carry
    most of the mass, as a trained draft head's output does."""
    rng = np.random.default_rng(seed + 11)
    z = sharp * rng.standard_normal((B, R, V))
    ids = np.arange(V)
    z = np.where((ids >= v_begin) & (ids < v_end), z, -np.inf)
    e = np.exp(z - z.max(axis=-1, keepdims=True))
    return (e / e.sum(axis=-1, keepdims=True)).astype(np.float32)


def draw_pool_uniforms(B: int, NQ: int, seed: int) -> np.ndarray:
    """u [B, NQ] fp32 in [0, 1): one uniform per pool distribution."""
    rng = np.random.default_rng(seed + 12)
    u = rng.random((B, NQ), dtype=np.float32)
    return np.minimum(u, np.nextafter(np.float32(1.0), np.float32(0.0)))
