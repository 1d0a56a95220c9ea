"""The whole verify step on the GPU: the host-buffer entry point against the three separate calls, and
the chained step (attention output fed to the head, logits fed to accept) against the chained oracle."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2510_25739_b200 import workloads as wl
from tests._util import bf16_to_torch, to_dev, torch_bf16_to_f64

pytestmark = pytest.mark.gpu


def _inputs(cfg, seed):
    a = wl.make_attn_inputs(cfg, seed, ragged=True)
    h = wl.make_head_inputs(cfg, seed)
    q = wl.random_probs(cfg, seed).astype(np.float32)
    u = wl.draw_uniforms(cfg, seed)
    return a, h, q, wl.draw_drafts(q, seed), u


@pytest.mark.parametrize("config_id,B", [(1, 1), (2, 3), (4, 2)])
def test_host_step_equals_the_three_calls(config_id, B):
    """hawk_verify_step_host (pinned host inputs, copies on two streams) gives bit for bit what the three
    entry points give on device-resident inputs; run twice to cover the reuse of the staging buffers."""
    import paper_2510_25739_b200 as hawk
    from paper_2510_25739_b200 import binding
    cfg = wl.config(config_id, B=B)
    a, h, q, drafts, u = _inputs(cfg, 40 + config_id)
    dev = "cuda"
    kc, vc, pl, w = (bf16_to_torch(a["k_cache"]), bf16_to_torch(a["v_cache"]), to_dev(a["prefix_len"]),
                     bf16_to_torch(h["w"]))
    max_pl = int(a["prefix_len"].max())
    host = dict(q=torch.from_numpy(a["q"].view(np.int16)).pin_memory(), x=torch.from_numpy(h["x"].view(np.int16)).pin_memory(),
                q_probs=torch.from_numpy(q).pin_memory(), draft=torch.from_numpy(drafts).pin_memory(),
                u_accept=torch.from_numpy(u["u_accept"]).pin_memory(), u_resample=torch.from_numpy(u["u_resample"]).pin_memory())
    h_len = torch.full((cfg.B,), -9, dtype=torch.int32).pin_memory()
    h_tok = torch.full((cfg.B,), -9, dtype=torch.int32).pin_memory()
    stage = {k: torch.empty_like(v, device=dev) for k, v in host.items()}
    attn_out = torch.empty((cfg.S, cfg.K, cfg.hidden), dtype=torch.bfloat16, device=dev)
    logits = torch.zeros((cfg.M, cfg.V), dtype=torch.float32, device=dev)
    d_len = torch.empty(cfg.B, dtype=torch.int32, device=dev); d_tok = torch.empty(cfg.B, dtype=torch.int32, device=dev)
    ws_a = torch.empty(max(16, hawk.verify_attn_workspace_bytes(cfg.S, cfg.K, cfg.H, cfg.H_kv, cfg.D, max_pl)),
                       dtype=torch.uint8, device=dev)
    ws_c = torch.empty(max(16, hawk.cfg_accept_workspace_bytes(cfg.B, cfg.K, cfg.V)), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    s = binding.StepHostArgs()
    s.B, s.K, s.H, s.H_kv, s.D, s.L_cap, s.max_prefix_len = cfg.B, cfg.K, cfg.H, cfg.H_kv, cfg.D, cfg.L_cap, max_pl
    s.V, s.v_begin, s.v_end, s.top_k = cfg.V, cfg.v_begin, cfg.v_end, cfg.top_k
    s.sm_scale, s.cfg_scale, s.temperature = float(a["sm_scale"]), cfg.cfg_scale, cfg.temperature
    for name in ("q", "x", "q_probs", "draft", "u_accept", "u_resample"):
        setattr(s, "h_" + name, host[name].data_ptr())
        setattr(s, "d_" + name, stage[name].data_ptr())
    s.h_accept_len, s.h_out_token = h_len.data_ptr(), h_tok.data_ptr()
    s.d_k_cache, s.d_v_cache, s.d_prefix_len, s.d_w = kc.data_ptr(), vc.data_ptr(), pl.data_ptr(), w.data_ptr()
    s.d_attn_out, s.d_logits, s.d_accept_len, s.d_out_token = (attn_out.data_ptr(), logits.data_ptr(),
                                                              d_len.data_ptr(), d_tok.data_ptr())
    s.d_attn_workspace, s.attn_workspace_bytes = ws_a.data_ptr(), ws_a.numel()
    s.d_accept_workspace, s.accept_workspace_bytes = ws_c.data_ptr(), ws_c.numel()
    s.d_status = status.data_ptr()

    # the three calls on device-resident copies of the same inputs
    want_attn = hawk.verify_attn(bf16_to_torch(a["q"]), kc, vc, pl, max_pl, float(a["sm_scale"]))
    want_logits = hawk.head_proj(bf16_to_torch(h["x"]), w, cfg.v_begin, cfg.v_end,
                                 logits=torch.zeros((cfg.M, cfg.V), dtype=torch.float32, device=dev))
    want_len, want_tok = hawk.cfg_accept(want_logits.view(cfg.S, cfg.K, cfg.V), to_dev(q), to_dev(drafts),
                                         to_dev(u["u_accept"]), to_dev(u["u_resample"]), cfg.v_begin, cfg.v_end,
                                         cfg.cfg_scale, cfg.temperature, cfg.top_k)
    for _ in range(2):
        h_len.fill_(-9); h_tok.fill_(-9)
        hawk.verify_step_host(s)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(attn_out.view(torch.int16), want_attn.view(torch.int16))
        assert torch.equal(logits[:, cfg.v_begin:cfg.v_end], want_logits[:, cfg.v_begin:cfg.v_end])
        assert torch.equal(h_len, want_len.cpu()) and torch.equal(h_tok, want_tok.cpu())


def test_refused_step_queues_nothing():
    """A step whose accept-stage argument is bad (temperature 0) is refused before the first copy: the staging
    buffers, the outputs and the status word keep their sentinels, and the stream has nothing to wait for."""
    import paper_2510_25739_b200 as hawk
    from paper_2510_25739_b200 import binding
    from paper_2510_25739_b200.binding import HawkError
    cfg = wl.config(1)
    dev = "cuda"
    a, h, q, drafts, u = _inputs(cfg, 77)
    host = dict(q=torch.from_numpy(a["q"].view(np.int16)).pin_memory(), x=torch.from_numpy(h["x"].view(np.int16)).pin_memory(),
                q_probs=torch.from_numpy(q).pin_memory(), draft=torch.from_numpy(drafts).pin_memory(),
                u_accept=torch.from_numpy(u["u_accept"]).pin_memory(), u_resample=torch.from_numpy(u["u_resample"]).pin_memory())
    stage = {k: torch.full_like(v, 21, device=dev) for k, v in host.items()}
    kc, vc, pl, w = (bf16_to_torch(a["k_cache"]), bf16_to_torch(a["v_cache"]), to_dev(a["prefix_len"]),
                     bf16_to_torch(h["w"]))
    attn_out = torch.full((cfg.S, cfg.K, cfg.hidden), 3.0, dtype=torch.bfloat16, device=dev)
    logits = torch.full((cfg.M, cfg.V), -7.0, dtype=torch.float32, device=dev)
    d_len = torch.full((cfg.B,), -9, dtype=torch.int32, device=dev)
    d_tok = torch.full((cfg.B,), -9, dtype=torch.int32, device=dev)
    h_len = torch.full((cfg.B,), -9, dtype=torch.int32).pin_memory()
    h_tok = torch.full((cfg.B,), -9, dtype=torch.int32).pin_memory()
    ws_a = torch.empty(max(16, hawk.verify_attn_workspace_bytes(cfg.S, cfg.K, cfg.H, cfg.H_kv, cfg.D, cfg.L)),
                       dtype=torch.uint8, device=dev)
    ws_c = torch.empty(max(16, hawk.cfg_accept_workspace_bytes(cfg.B, cfg.K, cfg.V)), dtype=torch.uint8, device=dev)
    status = torch.full((1,), 0, dtype=torch.int32, device=dev)
    s = binding.StepHostArgs()
    s.B, s.K, s.H, s.H_kv, s.D, s.L_cap, s.max_prefix_len = cfg.B, cfg.K, cfg.H, cfg.H_kv, cfg.D, cfg.L_cap, cfg.L
    s.V, s.v_begin, s.v_end, s.top_k = cfg.V, cfg.v_begin, cfg.v_end, cfg.top_k
    s.sm_scale, s.cfg_scale, s.temperature = float(a["sm_scale"]), cfg.cfg_scale, 0.0          # <- refused by the accept stage
    for name in ("q", "x", "q_probs", "draft", "u_accept", "u_resample"):
        setattr(s, "h_" + name, host[name].data_ptr())
        setattr(s, "d_" + name, stage[name].data_ptr())
    s.h_accept_len, s.h_out_token = h_len.data_ptr(), h_tok.data_ptr()
    s.d_k_cache, s.d_v_cache, s.d_prefix_len, s.d_w = kc.data_ptr(), vc.data_ptr(), pl.data_ptr(), w.data_ptr()
    s.d_attn_out, s.d_logits, s.d_accept_len, s.d_out_token = (attn_out.data_ptr(), logits.data_ptr(),
                                                              d_len.data_ptr(), d_tok.data_ptr())
    s.d_attn_workspace, s.attn_workspace_bytes = ws_a.data_ptr(), ws_a.numel()
    s.d_accept_workspace, s.accept_workspace_bytes = ws_c.data_ptr(), ws_c.numel()
    s.d_status = status.data_ptr()
    torch.cuda.synchronize()
    with pytest.raises(HawkError) as err:
        hawk.verify_step_host(s)
    assert err.value.code == 6                                   # parameter
    assert torch.cuda.current_stream().query()                   # nothing was queued behind the synchronize above
    torch.cuda.synchronize()
    for k, t in stage.items():
        assert (t == 21).all(), k                                # no input copy ran
    assert (attn_out == 3.0).all() and (logits == -7.0).all()
    assert (d_len == -9).all() and (d_tok == -9).all() and (h_len == -9).all() and (h_tok == -9).all()
    assert int(status.item()) == 0
    # and the same arguments with a valid temperature go through
    s.temperature = cfg.temperature
    hawk.verify_step_host(s)
    torch.cuda.synchronize()
    assert (h_len >= 0).all() and int(status.item()) == 0


def test_chained_step_against_chained_oracle():
    """Attention output used as the hidden state (hidden = H * D), its logits verified: GPU chain against
    oracle chain.  Rounding upstream (bf16 attention output) moves logits by parts in a thousand, so a
    sequence counts only if every decision the oracle took has a margin well above that."""
    import paper_2510_25739_b200 as hawk
    cfg = wl.config(2, B=16, L=300, top_k=200, cfg_scale=3.0)
    a, h, q_rand, _, u = _inputs(cfg, 91)
    # --- oracle chain
    o_attn = oracle.verify_attn(a["q"], a["k_cache"], a["v_cache"], a["prefix_len"], a["sm_scale"])
    x_bits = wl.f32_to_bf16_bits((o_attn * 8.0).astype(np.float32).reshape(cfg.M, cfg.hidden))   # scaled up: peaked logits
    o_logits = oracle.head_proj(x_bits, h["w"]).reshape(cfg.S, cfg.K, cfg.V)
    p, _ = oracle.target_probs_rows(o_logits, 0, cfg.V, cfg.cfg_scale, 1.0, cfg.top_k)
    q = wl.mix_q(p, wl.random_probs(cfg, 91), 0.6)
    drafts = wl.draw_drafts(q, 91)
    ora = oracle.cfg_accept(o_logits, q, drafts, u["u_accept"], u["u_resample"], 0, cfg.V, cfg.cfg_scale, 1.0, cfg.top_k)
    # --- GPU chain
    g_attn = hawk.verify_attn(bf16_to_torch(a["q"]), bf16_to_torch(a["k_cache"]), bf16_to_torch(a["v_cache"]),
                              to_dev(a["prefix_len"]), int(a["prefix_len"].max()), float(a["sm_scale"]))
    g_x = (g_attn.float() * 8.0).to(torch.bfloat16).view(cfg.M, cfg.hidden)      # the same scaling, by torch
    g_logits = hawk.head_proj(g_x, bf16_to_torch(h["w"]))
    g_len, g_tok = hawk.cfg_accept(g_logits.view(cfg.S, cfg.K, cfg.V), to_dev(q), to_dev(drafts), to_dev(u["u_accept"]),
                                   to_dev(u["u_resample"]), 0, cfg.V, cfg.cfg_scale, 1.0, cfg.top_k)
    torch.cuda.synchronize()
    lg = g_logits.cpu().numpy().reshape(cfg.S, cfg.K, cfg.V).astype(np.float64)
    rms = np.sqrt((o_logits.astype(np.float64) ** 2).mean())
    assert np.abs(lg - o_logits).max() <= 3e-2 * rms        # bf16 attention output, one more bf16 rounding of x
    g_len, g_tok = g_len.cpu().numpy(), g_tok.cpu().numpy()
    agree = wide = tok_checked = 0
    for b in range(cfg.B):
        olen = int(ora["accept_len"][b])
        examined = min(olen + 1, cfg.K)
        if (ora["accept_margin"][b, :examined] < 0.1).any():
            continue                                        # a decision that upstream rounding could move
        wide += 1
        agree += int(g_len[b] == olen)
        if g_len[b] != olen:
            continue
        # the correction token.  The GPU's logits differ from the oracle's by parts in a thousand, so its running
        # sums of the residual are shifted a little and the draw may land on a neighbouring id: the token must be
        # an id the oracle's residual gives mass to, and the oracle's draw point u * R must lie within 3 % of the
        # total mass of that id's slice of the oracle's running sums.
        if olen == cfg.K:
            assert g_tok[b] == -1 and ora["token"][b] == -1
            continue
        r = np.maximum(0.0, p[b, olen] - q[b, olen].astype(np.float64))
        R = r.sum()
        cdf = np.cumsum(r)
        t = float(u["u_resample"][b, olen]) * R
        tok = int(g_tok[b])
        assert 0 <= tok < cfg.V and r[tok] > 0.0, (b, tok)
        lo = cdf[tok - 1] if tok > 0 else 0.0
        assert lo - 3e-2 * R <= t <= cdf[tok] + 3e-2 * R, (b, tok, int(ora["token"][b]), lo / R, t / R, cdf[tok] / R)
        tok_checked += 1
    assert wide >= cfg.B // 2, "the case must leave sequences to compare"
    assert agree == wide, (agree, wide)
    assert tok_checked >= 1
    print(f"chained step: {wide} of {cfg.B} sequences with wide margins, all agree on accept_len; "
          f"{tok_checked} correction tokens consistent with the oracle's residual")
