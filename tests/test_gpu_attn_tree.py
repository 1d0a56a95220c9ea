"""GPU parity of hawk_verify_attn_tree (tree-masked attention) against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_25739_b200 import workloads as wl
from tests._util import bf16_to_torch, to_dev, torch_bf16_to_f64

pytestmark = pytest.mark.gpu

RTOL = 2e-2          # bf16 tolerance stated for attention outputs
ATOL_RMS = 1e-2      # plus this fraction of the output's rms (bf16 rounding of values near zero)


def _check(branching, B, H, H_kv, D, L, seed, ragged=True, masks=None):
    import paper_2510_25739_b200 as hawk
    if masks is None:
        tree = wl.make_tree(branching)
        masks = wl.tree_ancestor_masks(tree["child_begin"])
    N = len(masks)
    cfg = wl.config(1, B=B, K=N, H=H, H_kv=H_kv, D=D, L=L)
    a = wl.make_attn_inputs(cfg, seed, ragged=ragged)
    # slots past the block's rows must never influence the result
    kc = wl.bf16_bits_to_f32(a["k_cache"]); vc = wl.bf16_bits_to_f32(a["v_cache"])
    for s in range(cfg.S):
        kc[s, :, a["prefix_len"][s] + N:, :] = np.nan
        vc[s, :, a["prefix_len"][s] + N:, :] = np.nan
    a["k_cache"] = wl.f32_to_bf16_bits(np.nan_to_num(kc)); a["v_cache"] = wl.f32_to_bf16_bits(np.nan_to_num(vc))
    a["k_cache"][np.isnan(kc)] = 0x7FC0; a["v_cache"][np.isnan(vc)] = 0x7FC0
    want = oracle.verify_attn_tree(a["q"], a["k_cache"], a["v_cache"], a["prefix_len"], masks, a["sm_scale"])
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = hawk.verify_attn(bf16_to_torch(a["q"]), bf16_to_torch(a["k_cache"]), bf16_to_torch(a["v_cache"]),
                           to_dev(a["prefix_len"]), int(a["prefix_len"].max()), float(a["sm_scale"]),
                           dev_status=status, anc_mask=to_dev(masks.view(np.int64)))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = torch_bf16_to_f64(out)
    assert np.isfinite(got).all()
    rms = np.sqrt((want ** 2).mean())
    err = np.abs(got - want)
    bound = RTOL * np.abs(want) + ATOL_RMS * rms
    assert (err <= bound).all(), (err.max(), rms, np.unravel_index(np.argmax(err - bound), err.shape))


@pytest.mark.parametrize("branching,B,H,H_kv,D,L", [
    ((2,), 1, 2, 2, 64, 10),            # 3 nodes
    ((3, 2), 2, 4, 4, 64, 100),         # 10 nodes: two column tiles
    ((2, 2, 2), 1, 2, 2, 128, 70),      # 15 nodes, D = 128
    ((3, 2, 2), 2, 3, 3, 64, 300),      # 22 nodes: three column tiles
    ((3, 3, 2), 1, 2, 2, 64, 1200),     # 31 nodes: four column tiles, keys split over several shares
    ((3, 2, 2), 1, 2, 2, 128, 200),     # 22 nodes at D = 128: two items of 16 and 6 rows per head
    ((2, 2), 1, 8, 2, 64, 150),         # grouped-query: 4 heads x 7 nodes share a kv head
    ((3, 3, 3), 2, 2, 2, 64, 500),      # 40 nodes: mask bits past the 32nd, two items of 24 and 16 rows per head
    ((4, 3, 2), 1, 2, 2, 128, 333),     # 41 nodes at D = 128: two items of 24 and 17 rows per head
    ((2, 2, 2, 2, 2), 1, 3, 3, 64, 90), # 63 nodes
    ((7, 8), 2, 2, 1, 64, 1100),        # 64 nodes, two query heads per kv head: four items of 32 rows
    ((7, 8), 1, 2, 2, 128, 40),         # 64 nodes at D = 128: three items per head, the block longer than the prefix
])
def test_tree_shapes(branching, B, H, H_kv, D, L):
    _check(branching, B, H, H_kv, D, L, seed=500 + L)


def test_chain_mask_is_the_causal_kernel_bit_for_bit():
    import paper_2510_25739_b200 as hawk
    cfg = wl.config(2, B=2)
    a = wl.make_attn_inputs(cfg, 3)
    args = (bf16_to_torch(a["q"]), bf16_to_torch(a["k_cache"]), bf16_to_torch(a["v_cache"]),
            to_dev(a["prefix_len"]), cfg.L, float(a["sm_scale"]))
    masks = wl.chain_masks(cfg.K)
    o1 = hawk.verify_attn(*args)
    o2 = hawk.verify_attn(*args, anc_mask=to_dev(masks.view(np.int64)))
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16))


def test_config_shaped_tree():
    """22-node tree at the LlamaGen-XL shape (full-size launch, oracle on all of it: seconds)."""
    _check((3, 2, 2), 4, 20, 20, 64, 1144, seed=77, ragged=False)


@pytest.mark.parametrize("K,D", [(33, 64), (48, 128), (64, 64)])
def test_long_chains_against_the_causal_oracle(K, D):
    """A plain chain of more than 32 drafts through hawk_verify_attn (no mask argument): the kernel's own chain
    masks past the 32nd row, against the causal oracle."""
    import paper_2510_25739_b200 as hawk
    cfg = wl.config(1, B=1, K=K, H=2, H_kv=2, D=D, L=150)
    a = wl.make_attn_inputs(cfg, 600 + K, ragged=True)
    want = oracle.verify_attn(a["q"], a["k_cache"], a["v_cache"], a["prefix_len"], a["sm_scale"])
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = hawk.verify_attn(bf16_to_torch(a["q"]), bf16_to_torch(a["k_cache"]), bf16_to_torch(a["v_cache"]),
                           to_dev(a["prefix_len"]), int(a["prefix_len"].max()), float(a["sm_scale"]), dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = torch_bf16_to_f64(out)
    rms = np.sqrt((want ** 2).mean())
    assert (np.abs(got - want) <= RTOL * np.abs(want) + ATOL_RMS * rms).all()
