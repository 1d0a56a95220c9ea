"""The library built with index checks (-DHAWK_DEBUG) runs every kernel family on small and ragged cases without
raising HAWK_DEV_BOUNDS, gives the oracle's results, and leaves the guard words around every output untouched.

This is the stand-in for a memory checker, which cannot be run on the test machines: the debug build checks the
computed indices of the kernels (histogram bins, candidate slots, verdict and output positions, workspace slots,
cache rows, shared-memory stages) and reports through the call's status word instead of faulting; the harness adds
canaries before and after each output buffer.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_25739_b200 import binding, build
from paper_2510_25739_b200 import workloads as wl
from tests._util import bf16_to_torch, compare_accept, to_dev, torch_bf16_to_f64

pytestmark = pytest.mark.gpu

GUARD = 64          # guard elements on either side of an output


@pytest.fixture(scope="module")
def debug_lib():
    return build.build_debug_variant()


class Guarded:
    """An output tensor carved out of a larger buffer whose margins hold a sentinel."""

    def __init__(self, shape, dtype, sentinel):
        n = int(np.prod(shape))
        self.full = torch.full((n + 2 * GUARD,), sentinel, dtype=dtype, device="cuda")
        self.view = self.full[GUARD:GUARD + n].view(*shape)
        self.sentinel = sentinel

    def intact(self) -> bool:
        lo, hi = self.full[:GUARD], self.full[-GUARD:]
        if self.full.dtype.is_floating_point:
            return bool((lo.float() == float(self.sentinel)).all() and (hi.float() == float(self.sentinel)).all())
        return bool((lo == self.sentinel).all() and (hi == self.sentinel).all())


def _no_bounds(status):
    assert int(status.item()) & binding.DEV_BOUNDS == 0, "an index left its array"


@pytest.mark.parametrize("overrides,tree", [
    (dict(B=2, K=5, H=4, H_kv=4, D=64, L=333), None),              # equal shares, ragged prefixes
    (dict(B=1, K=3, H=8, H_kv=2, D=128, L=77), None),              # grouped-query heads, one warp per item
    (dict(B=8, K=5, H=20, H_kv=20, D=64, L=600), None),            # 320 items merged inside a block
    (dict(B=1, K=0, H=2, H_kv=2, D=64, L=140), (3, 3, 3)),         # a 40-node tree
])
def test_attention(overrides, tree, debug_lib):
    import paper_2510_25739_b200 as hawk
    masks = None
    if tree is not None:
        masks = wl.tree_ancestor_masks(wl.make_tree(tree)["child_begin"])
        overrides = dict(overrides, K=len(masks))
    cfg = wl.config(1, **overrides)
    a = wl.make_attn_inputs(cfg, 9100 + cfg.L, ragged=True)
    out = Guarded((cfg.S, cfg.K, cfg.hidden), torch.bfloat16, 3.0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    with binding.alternate_library(debug_lib):
        hawk.verify_attn(bf16_to_torch(a["q"]), bf16_to_torch(a["k_cache"]), bf16_to_torch(a["v_cache"]),
                         to_dev(a["prefix_len"]), int(a["prefix_len"].max()), float(a["sm_scale"]), out=out.view,
                         dev_status=status, anc_mask=None if masks is None else to_dev(masks.view(np.int64)))
        torch.cuda.synchronize()
    _no_bounds(status)
    assert int(status.item()) == 0 and out.intact()
    if masks is None:
        want = oracle.verify_attn(a["q"], a["k_cache"], a["v_cache"], a["prefix_len"], a["sm_scale"])
    else:
        want = oracle.verify_attn_tree(a["q"], a["k_cache"], a["v_cache"], a["prefix_len"], masks, a["sm_scale"])
    got = torch_bf16_to_f64(out.view)
    rms = np.sqrt((want ** 2).mean())
    assert (np.abs(got - want) <= 2e-2 * np.abs(want) + 1e-2 * rms).all()


@pytest.mark.parametrize("M,hidden,V,vb,ve", [
    (5, 192, 300, 0, 300),         # one block per tile, ragged
    (48, 1088, 1000, 4, 996),      # tiles split along the hidden dimension
    (333, 320, 700, 1, 699),       # pairs of blocks, one wide tile
    (600, 128, 1024, 0, 1024),     # pairs of blocks, 256-id tiles
])
def test_head(M, hidden, V, vb, ve, debug_lib):
    import paper_2510_25739_b200 as hawk
    rng = np.random.default_rng(9200 + M)
    x = wl.f32_to_bf16_bits(rng.standard_normal((M, hidden)).astype(np.float32))
    w = wl.f32_to_bf16_bits((rng.standard_normal((V, hidden)) * 0.02).astype(np.float32))
    logits = Guarded((M, V), torch.float32, -7.0)
    logits.view.fill_(-7.0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    with binding.alternate_library(debug_lib):
        hawk.head_proj(bf16_to_torch(x), bf16_to_torch(w), vb, ve, logits=logits.view, dev_status=status)
        torch.cuda.synchronize()
    assert int(status.item()) == 0 and logits.intact()
    got = logits.view.cpu().numpy()
    assert (got[:, :vb] == -7.0).all() and (got[:, ve:] == -7.0).all()
    want = oracle.head_proj(x, w, vb, ve, fill=-7.0).astype(np.float64)[:, vb:ve]
    rms = np.sqrt((want ** 2).mean())
    assert (np.abs(got[:, vb:ve] - want) <= 1e-5 * np.abs(want) + 1e-5 * rms).all()


@pytest.mark.parametrize("V,vb,ve,top_k,K,B,bonus", [
    (1000, 3, 999, 50, 3, 4, True),          # unaligned range
    (16384, 0, 16384, 2000, 5, 8, False),    # the XL-shaped rows
    (20000, 0, 20000, 300, 2, 2, False),     # 32 ids per thread
    (4096, 0, 4096, 100, 4, 70, True),       # 350 rows: verdicts marked unknown first, rows behind a rejection skipped
])
def test_accept(V, vb, ve, top_k, K, B, bonus, debug_lib):
    import paper_2510_25739_b200 as hawk
    cfg = wl.config(2, B=B, K=K, V=V, v_begin=vb, v_end=ve, top_k=top_k, cfg_scale=3.0, H=4, H_kv=4)
    seed = 9300 + V + K
    logits = wl.make_logits(cfg, seed, has_bonus_row=bonus)
    p, _ = oracle.target_probs_rows(logits, vb, ve, cfg.cfg_scale, cfg.temperature, top_k)
    q = wl.make_q(cfg, seed, np.nan_to_num(p[:, :K]))
    drafts = wl.draw_drafts(q, seed)
    u = wl.draw_uniforms(cfg, seed)
    ora = oracle.cfg_accept(logits, q, drafts, u["u_accept"], u["u_resample"], vb, ve, cfg.cfg_scale, cfg.temperature,
                            top_k, has_bonus_row=bonus)
    alen, tok = Guarded((B,), torch.int32, -77), Guarded((B,), torch.int32, -77)
    ws = Guarded((hawk.cfg_accept_workspace_bytes(B, K, V) // 4 + 4,), torch.int32, -77)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    with binding.alternate_library(debug_lib):
        hawk.cfg_accept(to_dev(logits), to_dev(q), to_dev(drafts), to_dev(u["u_accept"]), to_dev(u["u_resample"]), vb, ve,
                        cfg.cfg_scale, cfg.temperature, top_k, has_bonus_row=bonus, accept_len=alen.view,
                        out_token=tok.view, workspace=ws.view.view(torch.uint8), dev_status=status)
        torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert alen.intact() and tok.intact() and ws.intact()
    res = compare_accept(alen.view.cpu().numpy(), tok.view.cpu().numpy(), ora, K)
    assert not res["bad"], res["bad"][:5]


def test_tree_accept_and_pool(debug_lib):
    """A (3, 2, 2) tree verified through the debug build (accepted length, path and token against the oracle, in a
    call of more than 1.5 waves of rows too); then the cache / pool / draw chain."""
    import paper_2510_25739_b200 as hawk
    from tests.test_gpu_tree import _case
    with binding.alternate_library(debug_lib):
        _case(5, 4096, 0, 4096, 500, (3, 2, 2), seed=9400)          # asserts a zero status word and parity
        _case(24, 4096, 4, 4000, 300, (3, 2, 2), seed=9401)         # 528 rows: unreachable nodes return early
    tree = wl.make_tree((3, 2, 2))
    N, B, V = tree["N"], 3, 4096
    IW, VSD, K = 8, 2, 3
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    qv = to_dev(wl.make_head_probs(B, VSD, V, 0, V, 9402))
    qh = to_dev(wl.make_head_probs(B, K, V, 0, V, 9403))
    uu = to_dev(wl.draw_pool_uniforms(B, K * (1 + VSD), 9404))
    with binding.alternate_library(debug_lib):
        rows, tags = hawk.spec_cache_new(B, IW, VSD, V)
        for T in range(2 * IW + 3):
            hawk.spec_cache_put(qv, torch.full((B,), T, dtype=torch.int32, device="cuda"), rows, tags, IW)
        pos = torch.full((B,), 2 * IW + 2, dtype=torch.int32, device="cuda")
        pool, source = hawk.pool_build(qh, rows, tags, pos, IW, VSD)
        ntok = hawk.pool_sample(pool, uu, to_dev(tree["node_q"]), 0, V, dev_status=status)
        torch.cuda.synchronize()
    assert int(status.item()) == 0
    t = ntok.cpu().numpy()
    assert (t[:, 0] == 0).all() and ((t[:, 1:] >= 0) & (t[:, 1:] < V)).all()
    assert (pool.sum(dim=-1) - 1.0).abs().max() < 1e-3          # every pool row is one of the input distributions
    assert (source.cpu().numpy()[:, 1::(1 + VSD)] == 1).all()   # the depth-1 predictions were all found in the cache
