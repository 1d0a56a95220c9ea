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


def test_chain_mask_reproduces_causal_attention():
    rng = np.random.default_rng(5)
    K = 5
    q, kc, vc, pl = _rand_case(rng, 2, K, 3, 3, 16, 20, [12, 7])
    masks = np.array([(2 << i) - 1 for i in range(K)], np.uint32)
    np.testing.assert_array_equal(oracle.verify_attn_tree(q, kc, vc, pl, masks, 0.25),
                                  oracle.verify_attn(q, kc, vc, pl, 0.25))


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
