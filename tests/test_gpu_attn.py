"""GPU parity of hawk_verify_attn against the oracle (through the C ABI)."""
import json
import os
from pathlib import Path

import numpy as np
import pytest
import torch

import oracle
from paper_2510_25739_b200 import workloads as wl
from tests._util import bf16_to_torch, to_dev, torch_bf16_to_f64

pytestmark = pytest.mark.gpu

RTOL = 2e-2          # bf16 tolerance stated for attention outputs
ATOL_RMS = 1e-2      # plus this fraction of the output's rms (bf16 rounding of values near zero)
USED = {}            # test id -> largest (err - RTOL*|want|) / rms seen: how much of the rms term a case needs


def _check(cfg, seed, ragged=False, poison_tail=False):
    import paper_2510_25739_b200 as hawk
    a = wl.make_attn_inputs(cfg, seed, ragged=ragged)
    if poison_tail:     # slots past the block's rows must never influence the result
        kc = wl.bf16_bits_to_f32(a["k_cache"]); vc = wl.bf16_bits_to_f32(a["v_cache"])
        for s in range(cfg.S):
            kc[s, :, a["prefix_len"][s] + cfg.K:, :] = np.nan
            vc[s, :, a["prefix_len"][s] + cfg.K:, :] = np.nan
        a["k_cache"] = wl.f32_to_bf16_bits(kc); a["v_cache"] = wl.f32_to_bf16_bits(vc)
        a["k_cache"][np.isnan(kc)] = 0x7FC0; a["v_cache"][np.isnan(vc)] = 0x7FC0
    want = oracle.verify_attn(a["q"], a["k_cache"], a["v_cache"], a["prefix_len"], a["sm_scale"])
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = hawk.verify_attn(bf16_to_torch(a["q"]), bf16_to_torch(a["k_cache"]), bf16_to_torch(a["v_cache"]),
                           to_dev(a["prefix_len"]), int(a["prefix_len"].max()), float(a["sm_scale"]),
                           dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = torch_bf16_to_f64(out)
    assert np.isfinite(got).all()
    rms = np.sqrt((want ** 2).mean())
    err = np.abs(got - want)
    bound = RTOL * np.abs(want) + ATOL_RMS * rms
    assert (err <= bound).all(), (err.max(), rms, np.unravel_index(np.argmax(err - bound), err.shape))
    used = float(((err - RTOL * np.abs(want)) / rms).max())
    key = os.environ.get("PYTEST_CURRENT_TEST", "?").split("::")[-1].split(" ")[0]
    USED[key] = max(USED.get(key, -1.0), used)
    return err.max() / rms


SMALL = [
    # B, K, H, H_kv, D, L
    (1, 1, 1, 1, 64, 0),
    (1, 4, 2, 2, 64, 5),
    (2, 3, 4, 4, 64, 63),
    (1, 5, 3, 3, 64, 64),
    (2, 8, 2, 2, 64, 200),
    (1, 6, 2, 2, 128, 130),
    (1, 2, 8, 2, 64, 300),      # grouped-query: 4 query heads share a kv head
    (1, 5, 8, 1, 128, 77),      # 8 heads x 5 drafts > 16 rows: chunked
    (1, 9, 2, 2, 64, 500),      # K+1 = 9 rows (bonus position)
    (1, 16, 1, 1, 64, 100),
    (2, 4, 2, 2, 64, 1500),     # long enough to be split over several blocks
]


@pytest.mark.parametrize("B,K,H,H_kv,D,L", SMALL)
@pytest.mark.parametrize("ragged", [False, True])
def test_small_shapes(B, K, H, H_kv, D, L, ragged):
    cfg = wl.config(1, B=B, K=K, H=H, H_kv=H_kv, D=D, L=L)
    _check(cfg, 100 + L + K, ragged=ragged, poison_tail=True)


@pytest.mark.parametrize("config_id", [1, 2, 3, 4, 5])
def test_configs_full_size(config_id):
    cfg = wl.config(config_id)
    worst = _check(cfg, wl.seed_for(config_id), ragged=(config_id in (3, 5)))
    print(f"config {config_id}: max err / rms = {worst:.2e}")


@pytest.mark.parametrize("config_id,overrides", [
    (2, {}),                                        # 320 items of 36 tiles: four warps of one block per item
    (4, {}),                                        # 256 items, D = 128
    (1, dict(B=28, K=5, H=4, H_kv=4, L=300)),       # 224 items of 10 tiles: the smallest call that takes this shape
    (1, dict(B=37, K=8, H=6, H_kv=6, L=700)),       # 444 items: the largest
    (1, dict(B=19, K=3, H=12, H_kv=6, D=128, L=211)),  # 228 items, two query heads per kv head (6 of 8 rows used)
    (1, dict(B=63, K=1, H=6, H_kv=3, D=128, L=628)),   # one draft, grouped-query heads
])
def test_items_merged_inside_a_block_ragged(config_id, overrides):
    """Few long items of 8 rows: an item's four warps merge in shared memory; with ragged prefix lengths some of
    a short stream's four shares lie past its last visible key and contribute nothing."""
    cfg = wl.config(config_id, **overrides)
    _check(cfg, 700 + config_id + len(overrides), ragged=True, poison_tail=bool(overrides))


@pytest.mark.parametrize("L", wl.XL_PREFIX_SWEEP)
def test_xl_prefix_sweep(L):
    _check(wl.config(2, L=L), wl.seed_for(2, L))


def test_bitwise_repeatable():
    import paper_2510_25739_b200 as hawk
    cfg = wl.config(2)
    a = wl.make_attn_inputs(cfg, 1)
    args = (bf16_to_torch(a["q"]), bf16_to_torch(a["k_cache"]), bf16_to_torch(a["v_cache"]),
            to_dev(a["prefix_len"]), cfg.L, float(a["sm_scale"]))
    o1 = hawk.verify_attn(*args).clone()
    o2 = hawk.verify_attn(*args)
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16))


def test_zz_rms_term_actually_used():
    """Runs after the cases above (same module, defined last): reports how much of the rms term of the bound any
    case needed, stores the figures next to the other run outputs, and fails if the stated term is more than
    twice what the worst case uses (a bound that loose would hide a real error)."""
    assert USED, "no attention case ran before this one"
    worst_key = max(USED, key=USED.get)
    worst = USED[worst_key]
    print(f"rms term used: worst {worst:.3e} of rms ({worst_key}); stated {ATOL_RMS:.1e}")
    out = Path(os.environ.get("HAWK_TEST_OUT", Path(__file__).resolve().parent.parent / "gpurun_out"))
    if out.is_dir():
        (out / "attn_tolerance_used.json").write_text(json.dumps({"stated_atol_rms": ATOL_RMS, "worst": worst,
                                                                  "worst_case": worst_key, "cases": USED}, indent=1))
    assert worst <= ATOL_RMS
    assert ATOL_RMS <= 2.0 * max(worst, 0.0) + 1e-12, (worst, ATOL_RMS)
