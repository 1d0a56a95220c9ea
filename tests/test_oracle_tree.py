"""Pins of the oracle's verification of a candidate tree (several candidates per depth, each with its
own draft distribution; Sec. 4.2, Eq. "recur"; distribution preservation, App. A)."""
from pathlib import Path

import numpy as np
from scipy.stats import chi2

import oracle

GOLDEN = Path(__file__).parent / "golden" / "tree_worked_example.txt"


def _logits_of(p, B, N):
    """Same target p at every node, guidance scale 1: logits = log p in both streams."""
    with np.errstate(divide="ignore"):
        row = np.log(np.asarray(p, np.float64)).astype(np.float32)
    return np.broadcast_to(row, (2 * B, N, len(p))).copy()


def test_hand_computed_tree_walk():
    p = [2 / 5, 3 / 10, 1 / 5, 1 / 10]
    q = np.array([[[1 / 10, 1 / 5, 3 / 10, 2 / 5], [1 / 5, 1 / 10, 2 / 5, 3 / 10]]], np.float32)
    child_begin = np.array([1, 3, 4, 4, 4], np.int32)       # 0 -> {1, 2}, 1 -> {3}, 2 and 3 leaves
    node_q = np.array([0, 0, 1, 0], np.int32)
    n_cases = 0
    for line in GOLDEN.read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        left, right = line.split("->")
        cand, ures = left.split("|")
        c = cand.split()
        tok = np.array([[0, int(c[0]), int(c[2]), int(c[4])]], np.int32)
        ua = np.array([[0.0, float(c[1]), float(c[3]), float(c[5])]], np.float32)
        ur = np.array([[float(v) for v in ures.split()]], np.float32)
        want = [int(v) for v in right.split()]
        r = oracle.tree_accept(_logits_of(p, 1, 4), q, tok, node_q, child_begin, ua, ur, 0, 4, 1.0, 1.0, 0,
                               max_depth=2)
        assert [int(r["accept_len"][0]), int(r["token"][0]), *r["path"][0].tolist()] == want, line
        n_cases += 1
    assert n_cases == 8


def test_chain_shaped_tree_equals_chain_verification():
    """One child per node: the tree walk is the chain with a bonus row (two routines, one rule)."""
    rng = np.random.default_rng(3)
    B, K, V = 6, 4, 200
    logits = (rng.standard_normal((2 * B, K + 1, V)) * 2).astype(np.float32)
    z = rng.standard_normal((B, K, V))
    q = (np.exp(z) / np.exp(z).sum(-1, keepdims=True)).astype(np.float32)
    pt, _ = oracle.target_probs_rows(logits, 0, V, 2.0, 1.0, 50)
    drafts = pt[:, :K].argmax(-1).astype(np.int32)            # likely tokens, so that several levels pass
    drafts[::2, 2] = (drafts[::2, 2] + 1) % V                 # and some chains break in the middle
    ua = rng.random((B, K), dtype=np.float32)
    ur = rng.random((B, K + 1), dtype=np.float32)
    chain = oracle.cfg_accept(logits, q, drafts, ua, ur, 0, V, 2.0, 1.0, 50, has_bonus_row=True)
    N = K + 1
    tree = oracle.tree_accept(logits, q, np.concatenate([np.zeros((B, 1), np.int32), drafts], 1),
                              np.concatenate([[0], np.arange(K)]).astype(np.int32),
                              np.concatenate([np.arange(1, N + 1), [N]]).astype(np.int32)[: N + 1],
                              np.concatenate([np.zeros((B, 1), np.float32), ua], 1), ur, 0, V, 2.0, 1.0, 50)
    assert (tree["accept_len"] == chain["accept_len"]).all() and (tree["token"] == chain["token"]).all()
    assert chain["accept_len"].max() >= 2


def _one_level(p, qs, n_samples, seed):
    """Root with C candidates, candidate j drawn from qs[j]; returns emitted first token and accept_len."""
    rng = np.random.default_rng(seed)
    C, V = qs.shape
    N = C + 1
    B = n_samples
    tok = np.zeros((B, N), np.int32)
    for j in range(C):
        tok[:, j + 1] = rng.choice(V, size=B, p=qs[j] / qs[j].sum())
    ua = rng.random((B, N), dtype=np.float32)
    ur = rng.random((B, N), dtype=np.float32)
    child_begin = np.array([1] + [N] * N, np.int32)
    node_q = np.concatenate([[0], np.arange(C)]).astype(np.int32)
    r = oracle.tree_accept(_logits_of(p, B, N), np.broadcast_to(qs.astype(np.float32), (B, C, V)).copy(), tok,
                           node_q, child_begin, ua, ur, 0, V, 1.0, 1.0, 0, max_depth=1, diagnostics=False)
    first = np.where(r["accept_len"] > 0, tok[np.arange(B), np.maximum(r["path"][:, 0], 0)], r["token"])
    return first, r["accept_len"]


def _dists(V, C, seed):
    rng = np.random.default_rng(seed)
    p = rng.dirichlet(np.ones(V) * 0.5)
    qs = np.stack([0.5 * p + 0.5 * rng.dirichlet(np.ones(V) * 0.5) for _ in range(C)])
    return p, qs


def test_first_token_follows_p_with_three_different_draft_heads():
    V, C, n = 32, 3, 100_000
    p, qs = _dists(V, C, 11)
    first, _ = _one_level(p, qs, n, 12)
    counts = np.bincount(first, minlength=V)
    stat = ((counts - n * p) ** 2 / (n * p)).sum()
    assert stat < chi2.ppf(0.999, V - 1), stat


def test_all_rejected_rate_is_the_product_of_one_minus_acceptance():
    """r = prod_j (1 - alpha_j), alpha_j = sum_x min(p_j(x), q_j(x)) on the refined targets (App. A)."""
    V, C, n = 24, 3, 100_000
    p, qs = _dists(V, C, 21)
    pj, rate = p.copy(), 1.0
    for j in range(C):                                   # the recursion written out in numpy
        alpha = np.minimum(pj, qs[j]).sum()
        rate *= 1.0 - alpha
        res = np.maximum(pj - qs[j], 0.0)
        pj = res / res.sum()
    _, alen = _one_level(p, qs, n, 22)
    got = (alen == 0).mean()
    assert abs(got - rate) < 4 * np.sqrt(rate * (1 - rate) / n), (got, rate)


def test_special_cases():
    V = 16
    p, qs = _dists(V, 2, 31)
    # a candidate drawn from the target itself always passes
    first, alen = _one_level(p, np.stack([p, qs[0]]), 2000, 32)
    assert (alen == 1).all()
    # second head equal to the refined target: whatever the first head rejects, the second one passes
    res = np.maximum(p - qs[0], 0.0)
    _, alen = _one_level(p, np.stack([qs[0], res / res.sum()]), 5000, 33)
    assert (alen == 1).all()
    # draft heads that live where the target has no mass: every candidate is rejected, the draw is from p
    p2 = np.where(np.arange(V) % 2 == 0, p, 0.0); p2 /= p2.sum()
    q2 = np.where(np.arange(V) % 2 == 1, 1.0, 0.0); q2 /= q2.sum()
    first, alen = _one_level(p2, np.stack([q2, q2]), 20000, 34)
    assert (alen == 0).all() and (first % 2 == 0).all()
    counts = np.bincount(first, minlength=V)[::2]
    pe = p2[::2]
    assert ((counts - 20000 * pe) ** 2 / (20000 * pe)).sum() < chi2.ppf(0.999, len(pe) - 1)


def test_out_of_range_candidate_is_clamped_and_flagged():
    p = [0.25, 0.25, 0.25, 0.25]
    q = np.full((1, 1, 4), 0.25, np.float32)
    r = oracle.tree_accept(_logits_of(p, 1, 2), q, np.array([[0, 9]], np.int32), np.array([0, 0], np.int32),
                           np.array([1, 2, 2], np.int32), np.array([[0, 0.5]], np.float32),
                           np.array([[0.1, 0.1]], np.float32), 0, 4, 1.0, 1.0, 0)
    assert r["flags"] & oracle.FLAG_BAD_DRAFT and r["accept_len"][0] == 1
