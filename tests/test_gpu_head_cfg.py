"""GPU parity of the head with the guidance combine in its epilogue (hawk_head_proj_cfg) and of the accept
kernels that read its output (hawk_cfg_accept_guided, hawk_tree_accept_guided), through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_25739_b200 import workloads as wl
from tests._util import bf16_to_torch, compare_accept, to_dev

pytestmark = pytest.mark.gpu

RTOL = 1e-5          # the tolerance stated for logits, applied to the two logits a guided value is made of
ATOL_RMS = 1e-5


def _xw(B, rows, hidden, V, seed, x_std=1.0, w_std=0.02):
    rng = np.random.default_rng(seed)
    x = wl.f32_to_bf16_bits((rng.standard_normal((2 * B, rows, hidden)) * x_std).astype(np.float32))
    w = wl.f32_to_bf16_bits((rng.standard_normal((V, hidden)) * w_std).astype(np.float32))
    return x, w


def _guided_bound(x, w, B, s, T, vb, ve):
    """|error| allowed on a guided logit: the logit tolerance on lc and on lu, amplified by the combine
    (d guided / d lc = s / T, d guided / d lu = (1 - s) / T), plus the combine's own fp32 roundings."""
    hidden = x.shape[-1]
    plain = oracle.head_proj(x.reshape(-1, hidden), w, vb, ve, fill=0.0).astype(np.float64)
    plain = plain.reshape(2 * B, -1, w.shape[0])[..., vb:ve]
    rms = np.sqrt((plain ** 2).mean())
    e_c = RTOL * np.abs(plain[:B]) + ATOL_RMS * rms
    e_u = RTOL * np.abs(plain[B:]) + ATOL_RMS * rms
    return (abs(s) * e_c + abs(1 - s) * e_u) / T + 4 * 2.0 ** -24 * (abs(s) * np.abs(plain[:B]) + (abs(s) + 1) * np.abs(plain[B:])) / T


CASES = [
    # B, rows, hidden, V, v_begin, v_end, scale, temperature
    (1, 1, 64, 128, 0, 128, 3.0, 1.0),
    (2, 5, 128, 300, 0, 300, 7.5, 1.0),          # ragged vocab tile, 10 pairs in a half tile of 16
    (8, 5, 256, 1000, 4, 996, 3.0, 0.8),         # 40 pairs: the conditional box runs into unconditional rows
    (16, 8, 256, 520, 130, 400, 1.0, 1.0),       # 128 pairs: one full tile
    (13, 10, 192, 384, 0, 384, 0.0, 2.0),        # 130 pairs: two token tiles, the second nearly empty
    (30, 10, 320, 700, 1, 699, 3.0, 1.0),        # 300 pairs: three token tiles
    (3, 22, 1024, 2048, 0, 2048, 3.0, 1.0),      # tree-shaped rows, more k-blocks than stages
    (24, 8, 256, 1024, 0, 1024, 3.0, 1.0),       # 192 pairs = 384 rows: CTA pairs, all rows in one 384-column tile
    (25, 10, 192, 700, 3, 697, 7.5, 0.9),        # 250 pairs = 500 rows, ragged ids (512 accumulator columns)
    (13, 10, 128, 512, 0, 512, 3.0, 1.0),        # 130 pairs = 260 rows (320 columns: quarters of 80)
    (32, 8, 256, 1024, 0, 1024, 3.0, 1.0),       # 256 pairs = 512 rows: the CTA-pair kernel, two tiles of 128 pairs
    (40, 9, 128, 700, 5, 690, 7.5, 0.9),         # 360 pairs: CTA pairs, three ragged tiles
    (64, 8, 128, 5120, 0, 5120, 3.0, 1.0),       # 512 pairs, 80 tiles on 74 CTA pairs: two rounds
    (50, 10, 64, 5000, 3, 4995, 7.5, 0.8),       # 500 pairs, the same ragged
]


@pytest.mark.parametrize("B,rows,hidden,V,vb,ve,s,T", CASES)
def test_guided_head_matches_oracle(B, rows, hidden, V, vb, ve, s, T):
    import paper_2510_25739_b200 as hawk
    x, w = _xw(B, rows, hidden, V, seed=B * rows + V)
    want = oracle.head_proj_cfg(x, w, s, T, vb, ve, fill=-7.0)
    guided = torch.full((B, rows, V), -7.0, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    hawk.head_proj_cfg(bf16_to_torch(x), bf16_to_torch(w), s, T, vb, ve, guided=guided, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = guided.cpu().numpy()
    assert (got[..., :vb] == -7.0).all() and (got[..., ve:] == -7.0).all()
    err = np.abs(got[..., vb:ve].astype(np.float64) - want[..., vb:ve].astype(np.float64))
    bound = _guided_bound(x, w, B, s, T, vb, ve)
    assert (err <= bound).all(), (err.max(), np.unravel_index(np.argmax(err - bound), err.shape))


@pytest.mark.parametrize("B,rows,hidden,V,vb,ve,s,T", CASES[1:6])
def test_guided_head_is_the_plain_head_combined(B, rows, hidden, V, vb, ve, s, T):
    """Same accumulators, same three fp32 operations: combining hawk_head_proj's own output on the host
    gives hawk_head_proj_cfg's output bit for bit (the product s * (lc - lu) is exact in fp64, so fp64
    arithmetic rounded once reproduces the fused multiply-add except for double-rounding ties)."""
    import paper_2510_25739_b200 as hawk
    x, w = _xw(B, rows, hidden, V, seed=77 + V)
    dx, dw = bf16_to_torch(x), bf16_to_torch(w)
    plain = hawk.head_proj(dx.view(-1, hidden), dw, vb, ve).view(2 * B, rows, V)[..., vb:ve].cpu().numpy()
    guided = hawk.head_proj_cfg(dx, dw, s, T, vb, ve)[..., vb:ve].cpu().numpy()
    lc, lu = plain[:B], plain[B:]
    diff = (lc - lu).astype(np.float32)
    g = (np.float64(np.float32(s)) * diff.astype(np.float64) + lu.astype(np.float64)).astype(np.float32)
    if T != 1.0:
        g = (g / np.float32(T)).astype(np.float32)
    mismatch = g != guided
    assert mismatch.mean() < 1e-4                      # double rounding of the emulated fma, if any
    assert np.abs(g[mismatch] - guided[mismatch]).max(initial=0.0) <= np.abs(g).max() * 2.0 ** -22


@pytest.mark.parametrize("B,rows,hidden,V,vb,ve,s,T", [
    (2, 5, 2048, 2048, 0, 2048, 3.0, 1.0),       # 16 tiles of a 32-k-block hidden dimension: the plain head splits them
    (4, 6, 4096, 65536, 4, 8196, 3.0, 1.0),      # the 7B-shaped workload: 65 tiles, 64 k-blocks
    (1, 4, 1088, 1000, 4, 996, 7.5, 0.7),        # an odd number of k-blocks (17), ragged range
])
def test_guided_head_where_the_head_splits_the_hidden_dimension(B, rows, hidden, V, vb, ve, s, T):
    """Few tiles and hidden >= 1024: both forms of the head run as pairs of blocks that each sum half of the hidden
    dimension and add the halves (own + partner: one addition, the same in both forms).  The guided value recombined on
    the host from the plain logits is therefore hawk_head_proj_cfg's output bit for bit, as in the unsplit shapes."""
    import paper_2510_25739_b200 as hawk
    x, w = _xw(B, rows, hidden, V, seed=177 + V)
    dx, dw = bf16_to_torch(x), bf16_to_torch(w)
    plain = hawk.head_proj(dx.view(-1, hidden), dw, vb, ve).view(2 * B, rows, V)[..., vb:ve].cpu().numpy()
    guided = hawk.head_proj_cfg(dx, dw, s, T, vb, ve)[..., vb:ve].cpu().numpy()
    lc, lu = plain[:B], plain[B:]
    diff = (lc - lu).astype(np.float32)
    g = (np.float64(np.float32(s)) * diff.astype(np.float64) + lu.astype(np.float64)).astype(np.float32)
    if T != 1.0:
        g = (g / np.float32(T)).astype(np.float32)
    mismatch = g != guided
    assert mismatch.mean() < 1e-4                      # double rounding of the emulated fma, if any
    assert np.abs(g[mismatch] - guided[mismatch]).max(initial=0.0) <= np.abs(g).max() * 2.0 ** -22
    # and both agree with the oracle
    want = oracle.head_proj_cfg(x, w, s, T, vb, ve)[..., vb:ve].astype(np.float64)
    bound = _guided_bound(x, w, B, s, T, vb, ve)
    assert (np.abs(guided.astype(np.float64) - want) <= bound).all()


@pytest.mark.parametrize("config_id,B,has_bonus", [(1, 3, False), (2, 4, False), (2, 3, True), (4, 2, False)])
def test_two_call_form_equals_three_call_form(config_id, B, has_bonus):
    """head_proj_cfg + cfg_accept_guided return, bit for bit, what head_proj + cfg_accept return, and both
    agree with the oracle run on the GPU's guided logits."""
    import paper_2510_25739_b200 as hawk
    cfg = wl.config(config_id, B=B)
    rows = cfg.K + (1 if has_bonus else 0)
    seed = 500 + config_id
    x, w = _xw(cfg.B, rows, cfg.hidden, cfg.V, seed, w_std=0.02)
    dx, dw = bf16_to_torch(x), bf16_to_torch(w)
    q = wl.random_probs(cfg, seed).astype(np.float32)
    u = wl.draw_uniforms(cfg, seed)
    drafts = wl.draw_drafts(q, seed)
    dev_in = [to_dev(q), to_dev(drafts), to_dev(u["u_accept"]), to_dev(u["u_resample"])]
    logits = torch.full((2 * cfg.B, rows, cfg.V), float("nan"), dtype=torch.float32, device="cuda")
    hawk.head_proj(dx.view(-1, cfg.hidden), dw, cfg.v_begin, cfg.v_end, logits=logits.view(-1, cfg.V))
    len3, tok3 = hawk.cfg_accept(logits, *dev_in, cfg.v_begin, cfg.v_end, cfg.cfg_scale, cfg.temperature, cfg.top_k,
                                 has_bonus_row=has_bonus)
    guided = torch.full((cfg.B, rows, cfg.V), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    hawk.head_proj_cfg(dx, dw, cfg.cfg_scale, cfg.temperature, cfg.v_begin, cfg.v_end, guided=guided)
    len2, tok2 = hawk.cfg_accept_guided(guided, *dev_in, cfg.v_begin, cfg.v_end, cfg.top_k, has_bonus_row=has_bonus,
                                        dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0            # the NaN sentinels outside the valid range were never read
    assert torch.equal(len2, len3) and torch.equal(tok2, tok3)
    g = guided.cpu().numpy()
    ora = oracle.cfg_accept(np.concatenate([g, g]), q, drafts, u["u_accept"], u["u_resample"], cfg.v_begin, cfg.v_end,
                            1.0, 1.0, cfg.top_k, has_bonus_row=has_bonus)
    res = compare_accept(len2.cpu().numpy(), tok2.cpu().numpy(), ora, cfg.K)
    assert not res["bad"], res
    assert res["checked"] >= 1


def test_tree_two_call_form_equals_three_call_form():
    import paper_2510_25739_b200 as hawk
    tree = wl.make_tree((3, 2, 2))
    N, NQ = tree["N"], tree["NQ"]
    cfg = wl.config(2, B=3, K=N)
    seed = 611
    x, w = _xw(cfg.B, N, cfg.hidden, cfg.V, seed)
    dx, dw = bf16_to_torch(x), bf16_to_torch(w)
    qcfg = wl.config(2, B=3, K=NQ)
    q = wl.random_probs(qcfg, seed).astype(np.float32)
    tok = wl.draw_tree_tokens(q, tree, seed)
    uu = wl.draw_tree_uniforms(cfg.B, N, seed)
    common = [to_dev(q), to_dev(tok), to_dev(tree["node_q"]), to_dev(tree["child_begin"]), to_dev(uu["u_accept"]),
              to_dev(uu["u_resample"])]
    logits = hawk.head_proj(dx.view(-1, cfg.hidden), dw, cfg.v_begin, cfg.v_end).view(2 * cfg.B, N, cfg.V)
    a3 = hawk.tree_accept(logits, *common, cfg.v_begin, cfg.v_end, cfg.cfg_scale, cfg.temperature, cfg.top_k, max_depth=3)
    guided = hawk.head_proj_cfg(dx, dw, cfg.cfg_scale, cfg.temperature, cfg.v_begin, cfg.v_end)
    a2 = hawk.tree_accept_guided(guided, *common, cfg.v_begin, cfg.v_end, cfg.top_k, max_depth=3)
    torch.cuda.synchronize()
    for t3, t2 in zip(a3, a2):
        assert torch.equal(t3, t2)
    g = guided.cpu().numpy()
    ora = oracle.tree_accept(np.concatenate([g, g]), q, tok, tree["node_q"], tree["child_begin"], uu["u_accept"],
                             uu["u_resample"], cfg.v_begin, cfg.v_end, 1.0, 1.0, cfg.top_k, max_depth=3)
    alen, otok, path = (t.cpu().numpy() for t in a2)
    for b in range(cfg.B):
        if (ora["accept_margin"][b] < 1e-5).any():
            continue
        assert alen[b] == ora["accept_len"][b] and np.array_equal(path[b], ora["path"][b])
        if ora["resample_margin"][b] >= 1e-5:
            assert otok[b] == ora["token"][b]


def test_nonfinite_guided_input_is_flagged():
    import paper_2510_25739_b200 as hawk
    cfg = wl.config(1, B=2)
    seed = 9
    g = wl.make_logits(cfg, seed)[:cfg.B].copy()
    q = wl.random_probs(cfg, seed).astype(np.float32)
    u = wl.draw_uniforms(cfg, seed)
    drafts = wl.draw_drafts(q, seed)
    g[0, 0, cfg.v_begin + 3] = np.nan
    g[1, 1, cfg.v_begin + 5] = np.inf
    g[1, 0, cfg.v_begin + 7] = -np.inf            # a plain mask: no flag by itself
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    alen, tok = hawk.cfg_accept_guided(to_dev(g), to_dev(q), to_dev(drafts), to_dev(u["u_accept"]),
                                       to_dev(u["u_resample"]), cfg.v_begin, cfg.v_end, cfg.top_k, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 4                # HAWK_DEV_NONFINITE
    ora = oracle.cfg_accept(np.concatenate([g, g]), q, drafts, u["u_accept"], u["u_resample"], cfg.v_begin, cfg.v_end,
                            1.0, 1.0, cfg.top_k)
    assert ora["flags"] & oracle.FLAG_NONFINITE
    res = compare_accept(alen.cpu().numpy(), tok.cpu().numpy(), ora, cfg.K)
    assert not res["bad"], res


def test_argument_errors():
    import paper_2510_25739_b200 as hawk
    from paper_2510_25739_b200 import binding
    lib = hawk.load_library()
    P, st = binding._ptr, binding._stream()
    B, rows, hidden, V = 2, 3, 64, 128
    x, w = _xw(B, rows, hidden, V, 1)
    dx, dw = bf16_to_torch(x), bf16_to_torch(w)
    out = torch.empty((B, rows, V), dtype=torch.float32, device="cuda")
    f = lambda v: __import__("ctypes").c_float(v)
    assert lib.hawk_head_proj_cfg(None, P(dw), P(out), B, rows, hidden, V, 0, V, f(3.0), f(1.0), None, st) == 1
    assert lib.hawk_head_proj_cfg(P(dx), P(dw), P(out), -1, rows, hidden, V, 0, V, f(3.0), f(1.0), None, st) == 2
    assert lib.hawk_head_proj_cfg(P(dx), P(dw), P(out), B, rows, 96, V, 0, V, f(3.0), f(1.0), None, st) == 4
    assert lib.hawk_head_proj_cfg(P(dx), P(dw), P(out), B, rows, hidden, V, 0, V, f(3.0), f(0.0), None, st) == 6
    assert lib.hawk_head_proj_cfg(P(dx), P(dw), P(out), B, rows, hidden, V, 0, V, f(float("nan")), f(1.0), None, st) == 6
    assert lib.hawk_head_proj_cfg(P(dx), P(dw), P(out), 0, rows, hidden, V, 0, V, f(3.0), f(1.0), None, st) == 0
    torch.cuda.synchronize()
