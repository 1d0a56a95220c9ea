"""Speculation cache, spatial sampling pool and candidate tree (Sec. 4.2, Eqs. 1-5) as plain definitions.

Test infrastructure only, like the rest of this package.  The cache here is NOT the bounded buffer
of Eq. 2: it is the definition Cache(T + n, dv, d) read literally, an unbounded table keyed by the
raster position a prediction was made at and the depth of the head that made it.  That a buffer of
IW * VSD * (VSD + 1) / 2 slots returns the same rows is what the parity tests establish.

Pins: the number of predictions alive during a raster scan equals Eq. 2 (brute force); every
vertical pool row of speculation point T + n was made for exactly T + n (stamped predictions);
a hand-worked example under tests/golden; the candidate tree has prod(widths) leaves, every
root-to-leaf path is one element of the Cartesian product and no two paths coincide.
"""
from __future__ import annotations

import ctypes
import itertools

import numpy as np

from . import _c, _load, _p


def spec_cache_size(IW: int, VSD: int) -> int:
    """Eq. 2: IW * VSD * (VSD + 1) / 2 predictions per sequence."""
    return IW * (VSD * (VSD + 1)) // 2


class SpecCache:
    """Every vertical prediction ever made, per sequence: (position it was made at, depth) -> row.

    Eq. 1: the head of depth d, run at raster position T, predicts the token at T + IW * d.
    """

    def __init__(self, B: int, IW: int, VSD: int):
        self.B, self.IW, self.VSD = B, IW, VSD
        self.table = [dict() for _ in range(B)]

    def put(self, q_vert: np.ndarray, position: np.ndarray) -> None:
        """q_vert [B][VSD][V]: row d-1 is the depth-d prediction made at position[b] (< 0: none made)."""
        assert q_vert.shape[:2] == (self.B, self.VSD)
        for b in range(self.B):
            T = int(position[b])
            if T < 0:
                continue
            for d in range(1, self.VSD + 1):
                self.table[b][(T, d)] = np.array(q_vert[b, d - 1], copy=True)

    def lookup(self, b: int, target: int, dv: int):
        """Cache(target, dv, d = dv) of Eq. 3: the depth-dv prediction made dv rows above `target`."""
        return self.table[b].get((target - self.IW * dv, dv))

    def alive(self, b: int, T: int) -> int:
        """Predictions still needed when decoding stands at T: those whose target lies beyond T."""
        return sum(1 for (pos, d) in self.table[b] if pos + self.IW * d > T)


def pool_build(q_horiz: np.ndarray, cache: SpecCache, position: np.ndarray):
    """Eq. 5: Pool(T + n) = HorizSpec(T + n) followed by VertSpec(T + n), for n = 1 .. K.

    q_horiz [B][K][V]: row n-1 is the horizontal head's distribution for T + n (Eq. 4).
    Returns pool_q [B][K*(1+VSD)][V] (row (n-1)*(1+VSD) + j; j = 0 horizontal, j = dv vertical) and
    pool_source [B][K*(1+VSD)]: 0 horizontal, dv a cached vertical prediction, -dv none was cached
    and the horizontal distribution stands in.
    """
    B, K, V = q_horiz.shape
    VSD = cache.VSD
    width = 1 + VSD
    pool_q = np.empty((B, K * width, V), dtype=q_horiz.dtype)
    source = np.zeros((B, K * width), dtype=np.int32)
    for b in range(B):
        T = int(position[b])
        for n in range(1, K + 1):
            base = (n - 1) * width
            pool_q[b, base] = q_horiz[b, n - 1]
            for dv in range(1, VSD + 1):
                row = cache.lookup(b, T + n, dv) if T >= 0 else None
                if row is None:
                    pool_q[b, base + dv] = q_horiz[b, n - 1]
                    source[b, base + dv] = -dv
                else:
                    pool_q[b, base + dv] = row
                    source[b, base + dv] = dv
    return pool_q, source


def pool_sample(pool_q: np.ndarray, u: np.ndarray, v_begin: int, v_end: int):
    """One token per pool distribution (inverse CDF in ascending id); returns (row_token, margin)."""
    pool_q = _c(pool_q, np.float32)
    u = _c(u, np.float32)
    B, NQ, V = pool_q.shape
    assert u.shape == (B, NQ)
    tok = np.empty((B, NQ), dtype=np.int32)
    margin = np.empty((B, NQ), dtype=np.float64)
    lib = _load()
    lib.hawk_oracle_pool_sample.restype = None
    lib.hawk_oracle_pool_sample(_p(pool_q), _p(u), B * NQ, V, int(v_begin), int(v_end), _p(tok), _p(margin))
    return tok, margin


def candidate_tree(widths) -> dict:
    """Candidate tree as the Cartesian product of the per-position samples (Sec. 4.2).

    widths[n-1] candidates at speculation offset n.  A node is a prefix (j_1 .. j_m) of an element
    of the product; nodes are numbered breadth-first, prefixes of one length in lexicographic order,
    so the children of a node are consecutive.  node_q is the pool row of a node's last choice,
    (m - 1) * max(widths) + j_m.
    """
    stride = max(widths) if len(widths) else 0
    prefixes = [()]
    for m in range(1, len(widths) + 1):
        prefixes += list(itertools.product(*[range(w) for w in widths[:m]]))
    index = {p: i for i, p in enumerate(prefixes)}
    N = len(prefixes)
    child_begin = np.empty(N + 1, dtype=np.int32)
    node_q = np.zeros(N, dtype=np.int32)
    for i, p in enumerate(prefixes):
        m = len(p)
        child_begin[i] = index[p + (0,)] if m < len(widths) else N
        if m:
            node_q[i] = (m - 1) * stride + p[-1]
    child_begin[N] = N
    return dict(child_begin=child_begin, node_q=node_q, prefixes=prefixes, N=N, NQ=len(widths) * stride)


def node_tokens(row_token: np.ndarray, node_q: np.ndarray) -> np.ndarray:
    """node_token [B][N]: every node carries the sample of the pool row it stands for; the root carries 0."""
    out = row_token[:, node_q].astype(np.int32)
    out[:, 0] = 0
    return out
