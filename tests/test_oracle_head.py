"""Pins of the oracle's output-head projection (a plain matrix product)."""
import numpy as np

import oracle
from paper_2510_25739_b200 import workloads as wl


def test_matches_numpy_matmul():
    rng = np.random.default_rng(3)
    M, hidden, V = 5, 48, 37
    x = wl.f32_to_bf16_bits(rng.standard_normal((M, hidden)).astype(np.float32))
    w = wl.f32_to_bf16_bits((0.02 * rng.standard_normal((V, hidden))).astype(np.float32))
    got = oracle.head_proj(x, w)
    want = wl.bf16_bits_to_f32(x).astype(np.float64) @ wl.bf16_bits_to_f32(w).astype(np.float64).T
    assert got.dtype == np.float32
    np.testing.assert_allclose(got.astype(np.float64), want, rtol=6e-8, atol=1e-30)
    np.testing.assert_array_equal(got, want.astype(np.float32))     # one rounding, fp64 -> fp32


def test_identity_rows_return_the_hidden_state():
    rng = np.random.default_rng(4)
    M, hidden = 3, 16
    x = wl.f32_to_bf16_bits(rng.standard_normal((M, hidden)).astype(np.float32))
    w = wl.f32_to_bf16_bits(np.eye(hidden, dtype=np.float32))
    np.testing.assert_array_equal(oracle.head_proj(x, w), wl.bf16_bits_to_f32(x))


def test_only_the_valid_columns_are_written():
    rng = np.random.default_rng(5)
    M, hidden, V = 2, 8, 20
    x = wl.f32_to_bf16_bits(rng.standard_normal((M, hidden)).astype(np.float32))
    w = wl.f32_to_bf16_bits(rng.standard_normal((V, hidden)).astype(np.float32))
    full = oracle.head_proj(x, w)
    part = oracle.head_proj(x, w, 4, 11, fill=123.0)
    np.testing.assert_array_equal(part[:, 4:11], full[:, 4:11])
    assert (part[:, :4] == 123.0).all() and (part[:, 11:] == 123.0).all()


# ---- the head with the guidance combine applied to its output (generation settings of Sec. 5)
def _xw(rng, B, rows, hidden, V):
    x = wl.f32_to_bf16_bits(rng.standard_normal((2 * B, rows, hidden)).astype(np.float32))
    w = wl.f32_to_bf16_bits((0.05 * rng.standard_normal((V, hidden))).astype(np.float32))
    return x, w


def test_guided_head_special_scales():
    """Scale 0 returns the unconditional logits exactly, and a temperature divides them; scale 1 returns
    the conditional logits up to the rounding of the subtraction (lc - lu is not exact in fp32)."""
    rng = np.random.default_rng(6)
    B, rows, hidden, V = 2, 3, 32, 21
    x, w = _xw(rng, B, rows, hidden, V)
    plain = oracle.head_proj(x.reshape(-1, hidden), w).reshape(2 * B, rows, V)
    np.testing.assert_array_equal(oracle.head_proj_cfg(x, w, 0.0, 1.0), plain[B:])
    np.testing.assert_array_equal(oracle.head_proj_cfg(x, w, 0.0, 0.5), plain[B:] * np.float32(2.0))
    one = oracle.head_proj_cfg(x, w, 1.0, 1.0).astype(np.float64)
    ulp = 2.0 ** -23 * (np.abs(plain[:B]) + np.abs(plain[B:])).astype(np.float64)
    assert (np.abs(one - plain[:B]) <= ulp).all()
    assert not np.array_equal(one, plain[B:].astype(np.float64))


def test_guided_head_is_the_extrapolation_in_fp64():
    """Against the formula l = lu + s (lc - lu), then / T, on a numpy fp64 matrix product: the three fp32
    roundings allow 3 half-ulps of the largest term involved."""
    rng = np.random.default_rng(7)
    B, rows, hidden, V, s, T = 3, 2, 64, 50, 3.0, 0.7
    x, w = _xw(rng, B, rows, hidden, V)
    xf = wl.bf16_bits_to_f32(x).astype(np.float64).reshape(-1, hidden)
    l = (xf @ wl.bf16_bits_to_f32(w).astype(np.float64).T).reshape(2 * B, rows, V)
    want = (l[B:] + s * (l[:B] - l[B:])) / T
    bound = 4 * 2.0 ** -24 * (s * np.abs(l[:B]) + (s + 1) * np.abs(l[B:])) / T
    got = oracle.head_proj_cfg(x, w, s, T).astype(np.float64)
    assert (np.abs(got - want) <= bound).all()
    part = oracle.head_proj_cfg(x, w, s, T, 8, 40, fill=-7.0)
    np.testing.assert_array_equal(part[..., 8:40], got[..., 8:40].astype(np.float32))
    assert (part[..., :8] == -7.0).all() and (part[..., 40:] == -7.0).all()


def test_guided_head_then_accept_equals_head_then_guided_accept():
    """The two-call form decides on the same numbers as the three-call form: the target distribution
    from (head, combine inside the accept stage) equals the one from (combined head, accept stage told
    that nothing is left to combine), bit for bit."""
    rng = np.random.default_rng(8)
    B, rows, hidden, V, s, T, top_k = 2, 3, 32, 40, 3.0, 0.9, 7
    x, w = _xw(rng, B, rows, hidden, V)
    plain = oracle.head_proj(x.reshape(-1, hidden), w).reshape(2 * B, rows, V)
    guided = oracle.head_proj_cfg(x, w, s, T)
    p3, _ = oracle.target_probs_rows(plain, 0, V, s, T, top_k)
    p2, _ = oracle.target_probs_rows(np.concatenate([guided, guided]), 0, V, 1.0, 1.0, top_k)
    np.testing.assert_array_equal(p3, p2)
