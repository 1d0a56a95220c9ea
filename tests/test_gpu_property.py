"""Randomised small shapes (hypothesis): the CUDA path against the oracle on shapes no table lists."""
import numpy as np
import pytest
import torch
from hypothesis import given, settings, strategies as st

import oracle
from paper_2510_25739_b200 import workloads as wl
from tests._util import bf16_to_torch, compare_accept, to_dev, torch_bf16_to_f64

pytestmark = pytest.mark.gpu
SETTINGS = dict(max_examples=25, deadline=None, derandomize=True)


@settings(**SETTINGS)
@given(B=st.integers(1, 3), K=st.integers(1, 8), heads=st.sampled_from([(1, 1), (2, 2), (4, 2), (6, 3), (8, 1)]),
       D=st.sampled_from([64, 128]), L=st.integers(0, 300), seed=st.integers(0, 10_000))
def test_attention_random_shapes(B, K, heads, D, L, seed):
    import paper_2510_25739_b200 as hawk
    H, H_kv = heads
    cfg = wl.config(1, B=B, K=K, H=H, H_kv=H_kv, D=D, L=L)
    a = wl.make_attn_inputs(cfg, seed, ragged=True)
    want = oracle.verify_attn(a["q"], a["k_cache"], a["v_cache"], a["prefix_len"], a["sm_scale"])
    out = hawk.verify_attn(bf16_to_torch(a["q"]), bf16_to_torch(a["k_cache"]), bf16_to_torch(a["v_cache"]),
                           to_dev(a["prefix_len"]), int(a["prefix_len"].max()), float(a["sm_scale"]))
    got = torch_bf16_to_f64(out)
    rms = np.sqrt((want ** 2).mean())
    assert (np.abs(got - want) <= 2e-2 * np.abs(want) + 1e-2 * rms).all()


@settings(**SETTINGS)
@given(B=st.integers(1, 4), K=st.integers(1, 8), V=st.sampled_from([64, 1000, 4096, 16384]),
       top_mode=st.sampled_from(["none", "one", "some", "all"]), offset=st.sampled_from([0, 3, 4]),
       masked=st.booleans(), q_zeros=st.booleans(), bonus=st.booleans(), seed=st.integers(0, 10_000))
def test_accept_random_cases(B, K, V, top_mode, offset, masked, q_zeros, bonus, seed):
    import paper_2510_25739_b200 as hawk
    vb, ve = offset, V - (offset and 1)
    n = ve - vb
    top_k = {"none": 0, "one": 1, "some": max(1, n // 7), "all": n + 5}[top_mode]
    cfg = wl.config(2, B=B, K=K, V=V, v_begin=vb, v_end=ve, top_k=top_k, cfg_scale=2.5, H=4, H_kv=4)
    rng = np.random.default_rng(seed)
    logits = wl.make_logits(cfg, seed, has_bonus_row=bonus)
    if masked:                                            # -inf in one or both streams on a third of the ids
        hit = rng.random(logits.shape) < 0.33
        hit[..., :vb] = False; hit[..., ve:] = False
        logits[hit] = -np.inf
    p, flags = oracle.target_probs_rows(logits, vb, ve, cfg.cfg_scale, 1.0, top_k)
    q = wl.mix_q(np.nan_to_num(p[:, :K]), wl.random_probs(cfg, seed), 0.5)
    if q_zeros:                                           # a draft distribution with holes
        q[..., vb:ve][rng.random(q[..., vb:ve].shape) < 0.5] = 0.0
        q /= np.maximum(q.sum(-1, keepdims=True), 1e-30)
    drafts = wl.draw_drafts(np.where(q.sum(-1, keepdims=True) > 0, q, 1.0), seed)
    drafts = np.clip(drafts, vb, ve - 1).astype(np.int32)
    u = wl.draw_uniforms(cfg, seed)
    ora = oracle.cfg_accept(logits, q, drafts, u["u_accept"], u["u_resample"], vb, ve, cfg.cfg_scale, 1.0, top_k,
                            has_bonus_row=bonus)
    alen, tok = hawk.cfg_accept(to_dev(logits), to_dev(q), to_dev(drafts), to_dev(u["u_accept"]),
                                to_dev(u["u_resample"]), vb, ve, cfg.cfg_scale, 1.0, top_k, has_bonus_row=bonus)
    torch.cuda.synchronize()
    res = compare_accept(alen.cpu().numpy(), tok.cpu().numpy(), ora, K)
    assert not res["bad"], res["bad"][:5]
