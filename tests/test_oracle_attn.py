"""Pins of the oracle's attention (causal softmax attention of K draft queries over the cache)."""
import numpy as np
import pytest
from scipy.special import softmax

import oracle
from paper_2510_25739_b200 import workloads as wl


def _rand_case(rng, S, K, H, H_kv, D, L_cap, prefix):
    q = wl.f32_to_bf16_bits(rng.standard_normal((S, K, H, D)).astype(np.float32))
    kc = wl.f32_to_bf16_bits(rng.standard_normal((S, H_kv, L_cap, D)).astype(np.float32))
    vc = wl.f32_to_bf16_bits(rng.standard_normal((S, H_kv, L_cap, D)).astype(np.float32))
    return q, kc, vc, np.asarray(prefix, dtype=np.int32)


def _brute_force(q, kc, vc, prefix, scale):
    """Independent statement: masked score matrix, library softmax, matmul (vectorised per head)."""
    S, K, H, D = q.shape
    H_kv, L_cap = kc.shape[1], kc.shape[2]
    qf = wl.bf16_bits_to_f32(q).astype(np.float64)
    kf = wl.bf16_bits_to_f32(kc).astype(np.float64)
    vf = wl.bf16_bits_to_f32(vc).astype(np.float64)
    out = np.zeros((S, K, H * D))
    for s in range(S):
        for h in range(H):
            hk = h // (H // H_kv)
            scores = scale * qf[s, :, h, :] @ kf[s, hk].T            # [K, L_cap]
            j = np.arange(L_cap)[None, :]
            i = np.arange(K)[:, None]
            scores = np.where(j <= prefix[s] + i, scores, -np.inf)
            out[s, :, h * D:(h + 1) * D] = softmax(scores, axis=-1) @ vf[s, hk]
    return out


@pytest.mark.parametrize("S,K,H,H_kv,D,L_cap,prefix", [
    (2, 3, 2, 2, 8, 8, [5, 2]),
    (1, 1, 1, 1, 8, 1, [0]),
    (2, 2, 4, 2, 16, 9, [7, 0]),      # grouped-query: 2 query heads per KV head
    (1, 4, 3, 1, 8, 12, [8]),         # all query heads share one KV head
])
def test_matches_brute_force(S, K, H, H_kv, D, L_cap, prefix):
    rng = np.random.default_rng(7)
    q, kc, vc, pl = _rand_case(rng, S, K, H, H_kv, D, L_cap, prefix)
    got = oracle.verify_attn(q, kc, vc, pl, 1.0 / np.sqrt(D))
    want = _brute_force(q, kc, vc, pl, 1.0 / np.sqrt(D))
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)


def test_zero_queries_give_running_mean_of_values():
    rng = np.random.default_rng(8)
    S, K, H, D, L = 2, 3, 2, 8, 5
    q, kc, vc, pl = _rand_case(rng, S, K, H, H, D, L + K, [L, L - 2])
    q[:] = 0
    got = oracle.verify_attn(q, kc, vc, pl, 0.3)
    vf = wl.bf16_bits_to_f32(vc).astype(np.float64)
    for s in range(S):
        for i in range(K):
            n = pl[s] + i + 1
            for h in range(H):
                np.testing.assert_allclose(got[s, i, h * D:(h + 1) * D], vf[s, h, :n].mean(axis=0),
                                           rtol=1e-13, atol=1e-14)


def test_empty_prefix_single_query_returns_first_value_row():
    rng = np.random.default_rng(9)
    q, kc, vc, pl = _rand_case(rng, 1, 1, 2, 2, 8, 3, [0])
    got = oracle.verify_attn(q, kc, vc, pl, 0.35)
    vf = wl.bf16_bits_to_f32(vc).astype(np.float64)
    for h in range(2):
        np.testing.assert_array_equal(got[0, 0, h * 8:(h + 1) * 8], vf[0, h, 0])


def test_causality_later_block_rows_do_not_reach_earlier_queries():
    rng = np.random.default_rng(10)
    S, K, H, D, L = 1, 4, 2, 8, 6
    q, kc, vc, pl = _rand_case(rng, S, K, H, H, D, L + K, [L])
    base = oracle.verify_attn(q, kc, vc, pl, 0.35)
    for j in range(1, K):
        kc2, vc2 = kc.copy(), vc.copy()
        kc2[:, :, L + j:, :] = wl.f32_to_bf16_bits(np.full(1, 3.0, np.float32))[0]
        vc2[:, :, L + j:, :] = wl.f32_to_bf16_bits(np.full(1, -5.0, np.float32))[0]
        got = oracle.verify_attn(q, kc2, vc2, pl, 0.35)
        np.testing.assert_array_equal(got[:, :j], base[:, :j])          # rows i < j unchanged
        assert not np.array_equal(got[:, j:], base[:, j:])              # rows i >= j do change


def test_dominant_key_selects_its_value_row():
    S, K, H, D, L = 1, 1, 1, 8, 6
    qf = np.zeros((S, K, H, D), np.float32); qf[..., 0] = 8.0
    kf = np.zeros((S, H, L + K, D), np.float32); kf[0, 0, 3, 0] = 8.0     # score 64*scale at key 3
    rng = np.random.default_rng(11)
    vf = rng.standard_normal((S, H, L + K, D)).astype(np.float32)
    q, kc, vc = (wl.f32_to_bf16_bits(a) for a in (qf, kf, vf))
    got = oracle.verify_attn(q, kc, vc, np.array([L], np.int32), 1.0)
    np.testing.assert_allclose(got[0, 0], wl.bf16_bits_to_f32(vc)[0, 0, 3], atol=1e-25)   # other keys weigh exp(-64) each


def test_sm_scale_is_applied_to_the_scores():
    rng = np.random.default_rng(12)
    q, kc, vc, pl = _rand_case(rng, 1, 2, 1, 1, 8, 6, [4])
    a = oracle.verify_attn(q, kc, vc, pl, 0.5)
    b = _brute_force(q, kc, vc, pl, 0.5)
    c = _brute_force(q, kc, vc, pl, 1.0)
    np.testing.assert_allclose(a, b, rtol=1e-12)
    assert np.abs(a - c).max() > 1e-3
