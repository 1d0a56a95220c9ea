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
