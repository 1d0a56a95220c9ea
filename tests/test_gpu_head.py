"""GPU parity of hawk_head_proj (tcgen05 tensor-core path) against the oracle (through the C ABI)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_25739_b200 import workloads as wl
from tests._util import bf16_to_torch

pytestmark = pytest.mark.gpu

RTOL = 1e-5          # fp32 tolerance stated for logits
ATOL_RMS = 1e-5      # plus this fraction of the logits' rms (sums that cancel to near zero)


def _check(M, hidden, V, vb, ve, seed, x_std=1.0, w_std=0.02):
    import paper_2510_25739_b200 as hawk
    rng = np.random.default_rng(seed)
    x = wl.f32_to_bf16_bits((rng.standard_normal((M, hidden)) * x_std).astype(np.float32))
    w = wl.f32_to_bf16_bits((rng.standard_normal((V, hidden)) * w_std).astype(np.float32))
    want = oracle.head_proj(x, w, vb, ve, fill=-7.0)
    logits = torch.full((M, V), -7.0, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    hawk.head_proj(bf16_to_torch(x), bf16_to_torch(w), vb, ve, logits=logits, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = logits.cpu().numpy()
    # columns outside the range keep the sentinel
    assert (got[:, :vb] == -7.0).all() and (got[:, ve:] == -7.0).all()
    g = got[:, vb:ve].astype(np.float64); wv = want[:, vb:ve].astype(np.float64)
    rms = np.sqrt((wv ** 2).mean())
    err = np.abs(g - wv)
    bound = RTOL * np.abs(wv) + ATOL_RMS * rms
    assert (err <= bound).all(), (err.max(), rms, np.unravel_index(np.argmax(err - bound), err.shape))
    return err.max() / rms


SMALL = [
    # M, hidden, V, v_begin, v_end
    (1, 64, 128, 0, 128),
    (8, 128, 256, 0, 256),
    (5, 192, 300, 0, 300),         # ragged vocab tile, M not a multiple of 16
    (40, 256, 1000, 4, 996),       # range not aligned to the tile
    (100, 512, 520, 130, 400),
    (300, 256, 384, 0, 384),       # 257..511 rows: CTA pairs, one tile of all rows (two MMAs of half the columns)
    (384, 192, 700, 3, 697),       # the same at 384 rows with ragged 256-id tiles
    (500, 128, 512, 0, 512),       # ... and at 500 rows (512 accumulator columns)
    (333, 1856, 2475, 4, 2467),    # ... with 29 k-blocks and a ragged range
    (17, 1024, 2048, 0, 2048),     # more k-blocks than pipeline stages; few tiles: each split over two blocks along hidden
    (48, 1088, 1000, 4, 996),      # split along hidden with an odd number of k-blocks (17), ragged range
    (600, 320, 700, 1, 699),       # three token tiles, ragged both ways (from 512 rows on: the CTA-pair kernel)
    (512, 128, 256, 0, 256),       # CTA pairs: one tile of 256 ids x 256 rows per pair, two token tiles
    (1000, 192, 900, 3, 897),      # CTA pairs: ragged 256-id tiles, four token tiles of 256 rows (the last ragged)
    (513, 1024, 512, 0, 512),      # CTA pairs: three token tiles of 192 rows, more k-blocks than stages
    (1024, 128, 5120, 0, 5120),    # CTA pairs: 80 tiles on 74 pairs, a second, partly empty round
    (1000, 192, 5000, 7, 4990),    # ... ragged in both directions
]


@pytest.mark.parametrize("M,hidden,V,vb,ve", SMALL)
def test_small_shapes(M, hidden, V, vb, ve):
    _check(M, hidden, V, vb, ve, seed=M + V)


def test_identity_weight_returns_hidden_state():
    import paper_2510_25739_b200 as hawk
    rng = np.random.default_rng(1)
    hidden = 256
    x = wl.f32_to_bf16_bits(rng.standard_normal((24, hidden)).astype(np.float32))
    w = wl.f32_to_bf16_bits(np.eye(hidden, dtype=np.float32))
    got = hawk.head_proj(bf16_to_torch(x), bf16_to_torch(w)).cpu().numpy()
    np.testing.assert_array_equal(got, wl.bf16_bits_to_f32(x))


@pytest.mark.parametrize("config_id", [1, 2, 4])
def test_configs_full_size(config_id):
    cfg = wl.config(config_id)
    worst = _check(cfg.M, cfg.hidden, cfg.V, cfg.v_begin, cfg.v_end, wl.seed_for(config_id))
    print(f"config {config_id}: max err / rms = {worst:.2e}")


@pytest.mark.parametrize("config_id", [3, 5])
def test_large_configs_full_matrix(config_id):
    """Full-size launch of the two workloads with the most token rows (384 and 1024: the CTA-pair kernels), every
    logit compared with the oracle (its naive fp64 loops take a few seconds on the host cores)."""
    cfg = wl.config(config_id)
    worst = _check(cfg.M, cfg.hidden, cfg.V, cfg.v_begin, cfg.v_end, wl.seed_for(config_id))
    print(f"config {config_id}: max err / rms = {worst:.2e}")
