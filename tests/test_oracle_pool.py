"""Pins of the spatial-pool oracle (Sec. 4.2, Eqs. 1-5) against facts that do not come from it."""
from pathlib import Path

import numpy as np
import pytest

from oracle import spatial_pool as sp
from paper_2510_25739_b200 import workloads as wl

GOLDEN = Path(__file__).parent / "golden" / "pool_worked_example.txt"


def _stamp(pos, d, VSD, V):
    """A distribution that names the prediction it stands for: all mass on id pos * VSD + d - 1."""
    row = np.zeros(V, np.float32)
    row[pos * VSD + d - 1] = 1.0
    return row


def _run_history(steps, IW, VSD, V):
    cache = sp.SpecCache(1, IW, VSD)
    for pos in steps:
        qv = np.stack([_stamp(pos, d, VSD, V) for d in range(1, VSD + 1)])[None]
        cache.put(qv, np.array([pos], np.int32))
    return cache


def test_worked_example():
    IW, VSD, K, V = 4, 2, 2, 64
    steps = None
    n_cases = n_sizes = 0
    for line in GOLDEN.read_text().splitlines():
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("steps"):
            steps = [int(t) for t in line.split()[1:]]
            continue
        if line.startswith("size"):
            iw, vsd, want = (int(t) for t in line.split()[1:])
            assert sp.spec_cache_size(iw, vsd) == want
            n_sizes += 1
            continue
        head, *groups = [g.split() for g in line.split("|")]
        T = int(head[0])
        cache = _run_history(steps, IW, VSD, V)
        q_h = np.full((1, K, V), 1.0 / V, np.float32)
        pool_q, source = sp.pool_build(q_h, cache, np.array([T], np.int32))
        for n, group in enumerate(groups, start=1):
            base = (n - 1) * (1 + VSD)
            assert source[0, base] == 0 and np.array_equal(pool_q[0, base], q_h[0, n - 1])
            for dv, want in enumerate(group, start=1):
                if want == "-":
                    assert source[0, base + dv] == -dv
                    assert np.array_equal(pool_q[0, base + dv], q_h[0, n - 1])
                else:
                    pos, d = (int(t) for t in want.split(":"))
                    assert source[0, base + dv] == dv
                    assert np.array_equal(pool_q[0, base + dv], _stamp(pos, d, VSD, V))
        n_cases += 1
    assert n_cases == 3 and n_sizes == 3


@pytest.mark.parametrize("IW,VSD", [(4, 1), (5, 2), (8, 3), (3, 4)])
def test_alive_predictions_equal_eq2(IW, VSD):
    """Brute force: with a step at every raster position, the predictions whose target is still ahead
    number exactly IW * VSD * (VSD + 1) / 2 once the scan is VSD rows deep (Eq. 2), never more."""
    V = 4
    cache = sp.SpecCache(1, IW, VSD)
    peak = 0
    for T in range(IW * (2 * VSD + 3)):
        cache.put(np.zeros((1, VSD, V), np.float32), np.array([T], np.int32))
        alive = cache.alive(0, T)
        peak = max(peak, alive)
        if T >= IW * VSD:
            assert alive == sp.spec_cache_size(IW, VSD)
    assert peak == sp.spec_cache_size(IW, VSD)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_vertical_rows_point_at_the_speculation_point(seed):
    """Every vertical distribution in the pool of X was predicted FOR X (Sec. 4.2: results of different
    depths from different rows all point to the same inference point): predictions are stamped with
    their target P + IW * d at the time they are made, and read back from the pool."""
    rng = np.random.default_rng(seed)
    IW, VSD, K = 6, 3, 3
    V = IW * 12
    cache = sp.SpecCache(1, IW, VSD)
    T, made = 0, set()
    while T < IW * 9:
        qv = np.zeros((1, VSD, V), np.float32)
        for d in range(1, VSD + 1):
            tgt = T + IW * d
            if tgt < V:
                qv[0, d - 1, tgt] = 1.0
        cache.put(qv, np.array([T], np.int32))
        made.add(T)
        q_h = np.zeros((1, K, V), np.float32)
        q_h[0, :, 0] = 1.0  # the horizontal stand-in is recognisable: all mass on id 0
        pool_q, source = sp.pool_build(q_h, cache, np.array([T], np.int32))
        for n in range(1, K + 1):
            for dv in range(1, VSD + 1):
                row = pool_q[0, (n - 1) * (1 + VSD) + dv]
                src = T + n - IW * dv
                if src in made:
                    assert source[0, (n - 1) * (1 + VSD) + dv] == dv
                    assert row[T + n] == 1.0 and row.sum() == 1.0
                else:
                    assert source[0, (n - 1) * (1 + VSD) + dv] == -dv
                    assert row[0] == 1.0
        T += 1 + int(rng.integers(0, K + 1))  # accepted length of the step, then the corrected token


def test_candidate_tree_is_the_cartesian_product():
    widths = (3, 2, 2)
    t = sp.candidate_tree(widths)
    cb, N = t["child_begin"], t["N"]
    assert N == 1 + 3 + 6 + 12
    parent = np.full(N, -1)
    for i in range(N):
        parent[cb[i]:cb[i + 1]] = i
    leaves = [i for i in range(N) if cb[i] == cb[i + 1]]
    assert len(leaves) == 3 * 2 * 2
    paths = set()
    for leaf in leaves:
        rows, i = [], leaf
        while i > 0:
            rows.append(int(t["node_q"][i]))
            i = parent[i]
        rows.reverse()
        # the path picks one pool row per speculation offset, offset n from rows [(n-1)*3, (n-1)*3 + width)
        assert len(rows) == len(widths)
        for n, r in enumerate(rows):
            assert n * 3 <= r < n * 3 + widths[n]
        paths.add(tuple(rows))
    assert len(paths) == len(leaves)  # all distinct: the whole product, each element once
    # the seeded workload generator lays its trees out the same way
    g = wl.make_tree(widths)
    assert np.array_equal(g["child_begin"], cb) and np.array_equal(g["node_q"], t["node_q"])


def test_pool_sample_special_cases():
    V, vb, ve = 40, 3, 37
    q = np.zeros((1, 5, V), np.float32)
    q[0, 0, 11] = 0.7                      # point mass (un-normalised): always 11
    q[0, 1, 5] = 0.25; q[0, 1, 20] = 0.75  # boundary at 0.25
    q[0, 2, 5] = 0.25; q[0, 2, 20] = 0.75
    q[0, 3, 1] = 1.0; q[0, 3, 39] = 1.0    # mass only outside the valid ids: no token
    q[0, 4, vb:ve] = 1.0                   # uniform: id = vb + floor(u * 34)
    u = np.array([[0.999, 0.2499, 0.2501, 0.5, 0.5]], np.float32)
    tok, margin = sp.pool_sample(q, u, vb, ve)
    assert tok.tolist() == [[11, 5, 20, -1, vb + 17]]
    assert margin[0, 1] == pytest.approx(1e-4, rel=1e-2) and margin[0, 2] == pytest.approx(1e-4, rel=1e-2)
    tok0, _ = sp.pool_sample(q[:, 4:5], np.array([[0.0]], np.float32), vb, ve)
    tok1, _ = sp.pool_sample(q[:, 4:5], np.array([[np.nextafter(np.float32(1), np.float32(0))]], np.float32), vb, ve)
    assert tok0[0, 0] == vb and tok1[0, 0] == ve - 1


def test_pool_sample_follows_the_distribution():
    """Chi-square of 20000 draws from one 12-id distribution against that distribution."""
    rng = np.random.default_rng(7)
    V = 12
    q = rng.dirichlet(np.ones(V)).astype(np.float32)
    R = 20000
    u = rng.random((1, R), dtype=np.float32)
    tok, _ = sp.pool_sample(np.broadcast_to(q, (1, R, V)).copy(), u, 0, V)
    counts = np.bincount(tok[0], minlength=V)
    expect = q.astype(np.float64) / q.astype(np.float64).sum() * R
    chi2 = ((counts - expect) ** 2 / expect).sum()
    assert chi2 < 40.0  # 11 degrees of freedom: P(chi2 > 40) < 4e-5


def test_node_tokens_follow_node_q():
    t = sp.candidate_tree((2, 2))
    row_token = np.array([[10, 11, 12, 13]], np.int32)
    assert sp.node_tokens(row_token, t["node_q"]).tolist() == [[0, 10, 11, 12, 13, 12, 13]]
