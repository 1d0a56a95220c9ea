"""Pins of the oracle's tree attention: every tree node attends to the cached prefix and to the nodes
on its own path from the root (Sec. 4.2: candidates of a tree are verified in one forward pass)."""
import numpy as np
import pytest
from scipy.special import softmax

import oracle
from paper_2510_25739_b200 import workloads as wl
from tests.test_oracle_attn import _rand_case


def _brute_force(q, kc, vc, prefix, masks, scale):
    """Independent statement: boolean visibility matrix, library softmax, matmul."""
    S, N, H, D = q.shape
    H_kv, L_cap = kc.shape[1], kc.shape[2]
    qf = wl.bf16_bits_to_f32(q).astype(np.float64)
    kf = wl.bf16_bits_to_f32(kc).astype(np.float64)
    vf = wl.bf16_bits_to_f32(vc).astype(np.float64)
    out = np.zeros((S, N, H * D))
    for s in range(S):
        vis = np.zeros((N, L_cap), bool)
        vis[:, :prefix[s]] = True
        for i in range(N):
            for m in range(N):
                vis[i, prefix[s] + m] = bool((int(masks[i]) >> m) & 1)
        for h in range(H):
            hk = h // (H // H_kv)
            scores = np.where(vis, scale * qf[s, :, h, :] @ kf[s, hk].T, -np.inf)
            out[s, :, h * D:(h + 1) * D] = softmax(scores, axis=-1) @ vf[s, hk]
    return out


@pytest.mark.parametrize("branching,S,H,H_kv,D,prefix", [
    ((2,), 2, 2, 2, 8, [3, 0]),
    ((3, 2), 1, 4, 2, 16, [6]),
    ((2, 2, 2), 2, 1, 1, 8, [9, 4]),
    ((3, 2, 2), 1, 2, 1, 8, [5]),
    ((3, 3, 3), 1, 2, 2, 8, [7]),          # 40 nodes: masks past the 32nd bit
    ((4, 3, 2), 2, 2, 1, 8, [3, 11]),      # 41 nodes
    ((2, 2, 2, 2, 2), 1, 1, 1, 8, [2]),    # 63 nodes
    ((7, 8), 1, 2, 2, 8, [0]),             # 64 nodes, no prefix at all
])
def test_matches_brute_force(branching, S, H, H_kv, D, prefix):
    tree = wl.make_tree(branching)
    N = tree["N"]
    masks = wl.tree_ancestor_masks(tree["child_begin"])
    rng = np.random.default_rng(N + D)
    q, kc, vc, pl = _rand_case(rng, S, N, H, H_kv, D, max(prefix) + N + 2, prefix)
    got = oracle.verify_attn_tree(q, kc, vc, pl, masks, 0.3)
    np.testing.assert_allclose(got, _brute_force(q, kc, vc, pl, masks, 0.3), rtol=1e-12, atol=1e-13)


def test_ancestor_masks_of_a_known_tree():
    # 0 -> {1, 2}; 1 -> {3, 4}; 2 -> {5, 6}
    masks = wl.tree_ancestor_masks(wl.make_tree((2, 2))["child_begin"])
    assert masks.tolist() == [0b1, 0b11, 0b101, 0b1011, 0b10011, 0b100101, 0b1000101]


@pytest.mark.parametrize("K", [5, 33, 40, 64])
def test_chain_mask_reproduces_causal_attention(K):
    rng = np.random.default_rng(5 + K)
    q, kc, vc, pl = _rand_case(rng, 2, K, 3, 3, 16, 15 + K, [12, 7])
    masks = wl.chain_masks(K)
    assert masks.dtype == np.uint64 and int(masks[-1]) == (1 << K) - 1
    np.testing.assert_array_equal(oracle.verify_attn_tree(q, kc, vc, pl, masks, 0.25),
                                  oracle.verify_attn(q, kc, vc, pl, 0.25))


def test_high_mask_bits_matter():
    """A 40-node tree: clearing bit 35 of node 39's mask (an ancestor past the 32nd row) changes node 39 and nothing
    else; a mask type narrower than 64 bits would drop that bit silently."""
    tree = wl.make_tree((3, 3, 3))
    masks = wl.tree_ancestor_masks(tree["child_begin"])
    N = tree["N"]
    assert N == 40
    node = 39
    anc = [m for m in range(N) if (int(masks[node]) >> m) & 1]
    assert max(a for a in anc if a != node) >= 12        # its parent is a depth-2 node
    # give node 39 one more visible row past bit 32 instead: row 35 (not an ancestor)
    assert not (int(masks[node]) >> 35) & 1
    rng = np.random.default_rng(11)
    q, kc, vc, pl = _rand_case(rng, 1, N, 1, 1, 8, 3 + N, [3])
    base = oracle.verify_attn_tree(q, kc, vc, pl, masks, 0.4)
    m2 = masks.copy()
    m2[node] = np.uint64(int(m2[node]) | (1 << 35))
    other = oracle.verify_attn_tree(q, kc, vc, pl, m2, 0.4)
    assert not np.array_equal(base[:, node], other[:, node])
    keep = [i for i in range(N) if i != node]
    np.testing.assert_array_equal(base[:, keep], other[:, keep])
    np.testing.assert_allclose(other, _brute_force(q, kc, vc, pl, m2, 0.4), rtol=1e-12, atol=1e-13)


def test_rows_off_the_path_do_not_reach_a_node():
    """Changing the key/value rows of nodes that are not ancestors leaves a node's output bit-identical."""
    tree = wl.make_tree((2, 2))
    masks = wl.tree_ancestor_masks(tree["child_begin"])
    N = tree["N"]
    rng = np.random.default_rng(9)
    q, kc, vc, pl = _rand_case(rng, 1, N, 2, 2, 8, 4 + N, [4])
    base = oracle.verify_attn_tree(q, kc, vc, pl, masks, 0.5)
    node = 3                                             # path 0 -> 1 -> 3
    kc2, vc2 = kc.copy(), vc.copy()
    for m in range(N):
        if not (int(masks[node]) >> m) & 1:
            kc2[:, :, 4 + m, :] = wl.f32_to_bf16_bits(rng.standard_normal((1, 2, 8)).astype(np.float32) * 9)
            vc2[:, :, 4 + m, :] = wl.f32_to_bf16_bits(rng.standard_normal((1, 2, 8)).astype(np.float32) * 9)
    other = oracle.verify_attn_tree(q, kc2, vc2, pl, masks, 0.5)
    np.testing.assert_array_equal(base[:, node], other[:, node])
    assert not np.array_equal(base[:, 4], other[:, 4])   # node 4's own row was among those changed


def test_root_alone_sees_prefix_and_itself():
    rng = np.random.default_rng(2)
    q, kc, vc, pl = _rand_case(rng, 1, 1, 1, 1, 8, 3, [0])
    out = oracle.verify_attn_tree(q, kc, vc, pl, np.array([1], np.uint32), 1.0)
    np.testing.assert_allclose(out[0, 0], wl.bf16_bits_to_f32(vc)[0, 0, 0].astype(np.float64), rtol=0, atol=0)
