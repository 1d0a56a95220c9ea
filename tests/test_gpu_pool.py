"""GPU parity of the speculation cache, the sampling pool and the candidate draw (Sec. 4.2, Eqs. 1-5)
against the plain-definition oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from oracle import spatial_pool as sp
from paper_2510_25739_b200 import workloads as wl
from tests._util import to_dev

pytestmark = pytest.mark.gpu
TOL = 1e-5


def _check_tokens(node_token, ora_row_token, margin, node_q):
    """Bit-exact tokens except where the draw lies within TOL (fraction of the row's mass) of a CDF boundary."""
    want = sp.node_tokens(ora_row_token, node_q)
    exempt = margin[:, node_q] < TOL
    exempt[:, 0] = False
    bad = (node_token != want) & ~exempt
    assert not bad.any(), (np.argwhere(bad)[:5], node_token[bad][:5], want[bad][:5])
    return int(exempt.sum()), int((~exempt).sum())


@pytest.mark.parametrize("B,IW,VSD,K,V,vb,ve", [
    (3, 4, 2, 2, 64, 0, 64),
    (4, 8, 3, 3, 1001, 5, 998),         # rows that cannot be copied 16 bytes at a time
    (2, 6, 1, 4, 16384, 0, 16384),
    (5, 5, 4, 2, 4100, 4, 4100),
    (2, 32, 2, 3, 16384, 0, 16384),     # a 32 x 32 token image
    (1, 3, 8, 1, 40000, 0, 32768),      # deepest cache, widest id range
])
def test_steps_match_oracle(B, IW, VSD, K, V, vb, ve):
    import paper_2510_25739_b200 as hawk
    rng = np.random.default_rng(1000 + IW * VSD + V)
    assert hawk.spec_cache_slots(IW, VSD) == sp.spec_cache_size(IW, VSD)
    rows, tags = hawk.spec_cache_new(B, IW, VSD, V)
    cache = sp.SpecCache(B, IW, VSD)
    tree = sp.candidate_tree((1 + VSD,) * K)
    node_q = tree["node_q"]
    position = rng.integers(0, IW, size=B).astype(np.int32)
    position[0] = 0
    n_steps = 0
    n_vertical = n_standin = n_exempt = n_checked = 0
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    while position.min() < IW * (VSD + 2) and n_steps < 40:
        seed = 7000 + 13 * n_steps
        q_vert = wl.make_head_probs(B, VSD, V, vb, ve, seed)
        q_horiz = wl.make_head_probs(B, K, V, vb, ve, seed + 1)
        u = wl.draw_pool_uniforms(B, K * (1 + VSD), seed)
        d_pos = to_dev(position)
        # the heads ran at `position`: keep the vertical predictions, then build the pools of position + 1 ..
        cache.put(q_vert, position)
        hawk.spec_cache_put(to_dev(q_vert), d_pos, rows, tags, IW)
        want_q, want_src = sp.pool_build(q_horiz, cache, position)
        pool_q, source = hawk.pool_build(to_dev(q_horiz), rows, tags, d_pos, IW, VSD)
        torch.cuda.synchronize()
        assert np.array_equal(source.cpu().numpy(), want_src)
        assert np.array_equal(pool_q.cpu().numpy(), want_q)          # copies: bit-exact
        n_vertical += int((want_src > 0).sum())
        n_standin += int((want_src < 0).sum())
        ora_tok, margin = sp.pool_sample(want_q, u, vb, ve)
        node_token = hawk.pool_sample(pool_q, to_dev(u), to_dev(node_q), vb, ve, dev_status=status)
        torch.cuda.synchronize()
        e, c = _check_tokens(node_token.cpu().numpy(), ora_tok, margin, node_q)
        n_exempt += e
        n_checked += c
        position = (position + 1 + rng.integers(0, K + 1, size=B)).astype(np.int32)
        n_steps += 1
    assert int(status.item()) == 0
    assert n_vertical > 0 and n_standin > 0        # both kinds of pool row were exercised
    assert n_exempt <= max(3, n_checked // 10)


def test_bounded_cache_never_loses_a_live_prediction():
    """A step at every position for many rows: the Eq. 2 sized buffer serves every lookup the unbounded
    table of the oracle serves (rows are one-hot stamps of their target, so a stale row would show)."""
    import paper_2510_25739_b200 as hawk
    B, IW, VSD, K = 2, 5, 3, 2
    V = IW * 12 + 4
    rows, tags = hawk.spec_cache_new(B, IW, VSD, V)
    cache = sp.SpecCache(B, IW, VSD)
    for T in range(IW * 9):
        position = np.array([T, T], np.int32)
        q_vert = np.zeros((B, VSD, V), np.float32)
        for d in range(1, VSD + 1):
            q_vert[:, d - 1, (T + IW * d) % V] = 1.0
        q_horiz = np.zeros((B, K, V), np.float32)
        q_horiz[:, :, V - 1] = 1.0
        cache.put(q_vert, position)
        hawk.spec_cache_put(to_dev(q_vert), to_dev(position), rows, tags, IW)
        want_q, want_src = sp.pool_build(q_horiz, cache, position)
        pool_q, source = hawk.pool_build(to_dev(q_horiz), rows, tags, to_dev(position), IW, VSD)
        assert np.array_equal(source.cpu().numpy(), want_src)
        assert np.array_equal(pool_q.cpu().numpy(), want_q)
        if T >= IW * VSD:
            assert (want_src[:, 1::1 + VSD] > 0).all() and (want_src >= 0).all()
    assert int((tags.cpu().numpy() >= 0).sum()) == B * sp.spec_cache_size(IW, VSD)   # every slot in use


def test_clear_and_negative_position():
    import paper_2510_25739_b200 as hawk
    B, IW, VSD, K, V = 2, 4, 2, 2, 64
    rows, tags = hawk.spec_cache_new(B, IW, VSD, V)
    q_vert = wl.make_head_probs(B, VSD, V, 0, V, 1)
    q_horiz = wl.make_head_probs(B, K, V, 0, V, 2)
    hawk.spec_cache_put(to_dev(q_vert), to_dev(np.array([1, -1], np.int32)), rows, tags, IW)
    t = tags.cpu().numpy()
    assert (t[1] == -1).all() and (t[0] >= 0).sum() == VSD
    assert t[0, hawk.spec_cache_slot(IW, VSD, 1, 1)] == 1 and t[0, hawk.spec_cache_slot(IW, VSD, 1, 2)] == 1
    pool_q, source = hawk.pool_build(to_dev(q_horiz), rows, tags, to_dev(np.array([4, 4], np.int32)), IW, VSD)
    src = source.cpu().numpy()     # X = 5: one row above is position 1 (made, sequence 0 only); X = 6: nothing
    assert src.tolist() == [[0, 1, -2, 0, -1, -2], [0, -1, -2, 0, -1, -2]]
    assert np.array_equal(pool_q[0, 1].cpu().numpy(), q_vert[0, 0])
    hawk.spec_cache_clear(tags, IW, VSD)
    _, source = hawk.pool_build(to_dev(q_horiz), rows, tags, to_dev(np.array([4, 4], np.int32)), IW, VSD)
    assert (source.cpu().numpy()[:, 1] == -1).all()
    _, none = hawk.pool_build(to_dev(q_horiz), rows, tags, to_dev(np.array([4, 4], np.int32)), IW, VSD,
                              with_source=False)
    assert none is None


def test_sample_special_rows_and_bad_node_q():
    import paper_2510_25739_b200 as hawk
    V, vb, ve = 4096, 8, 4000
    q = np.zeros((1, 4, V), np.float32)
    q[0, 0, 77] = 3.0                       # un-normalised point mass
    q[0, 1, 2] = 1.0; q[0, 1, 4090] = 1.0   # mass only outside the valid ids
    q[0, 2, vb:ve] = 1.0                    # uniform
    q[0, 3, 100] = 0.5; q[0, 3, 200] = -5.0; q[0, 3, 300] = 0.5    # a negative weight counts as zero
    u = np.array([[0.9, 0.5, 0.2501, 0.75]], np.float32)
    node_q = np.array([0, 0, 1, 2, 3, 9, -1], np.int32)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tok = hawk.pool_sample(to_dev(q), to_dev(u), to_dev(node_q), vb, ve, dev_status=status).cpu().numpy()
    ora, _ = sp.pool_sample(q, u, vb, ve)
    assert ora.tolist() == [[77, -1, vb + 998, 300]]
    assert tok[0, :5].tolist() == [0, 77, -1, vb + 998, 300]
    assert tok[0, 5] == 300 and tok[0, 6] == 77        # clamped to the nearest row
    assert int(status.item()) == 16                    # HAWK_DEV_BAD_TREE


def test_draw_feeds_tree_accept_like_the_oracle():
    """One whole drafting + verification iteration per step on synthetic heads: cache, pool, draw, tree
    verification, position advanced by the accepted length + 1."""
    import paper_2510_25739_b200 as hawk
    B, IW, VSD, K, V, vb, ve, top_k, s = 6, 6, 1, 3, 4096, 0, 4096, 300, 3.0
    tree = sp.candidate_tree((1 + VSD,) * K)
    N, NQ = tree["N"], tree["NQ"]
    node_q, child_begin = tree["node_q"], tree["child_begin"]
    rows, tags = hawk.spec_cache_new(B, IW, VSD, V)
    cache = sp.SpecCache(B, IW, VSD)
    position = np.zeros(B, np.int32)
    lens = []
    for step in range(12):
        seed = 9100 + step
        cfg = wl.config(2, B=B, K=N, V=V, v_begin=vb, v_end=ve, top_k=top_k, cfg_scale=s, H=4, H_kv=4)
        logits = wl.make_logits(cfg, seed)
        p, _ = oracle.target_probs_rows(logits, vb, ve, s, 1.0, top_k)
        # heads that resemble the target at the root, so that some candidates pass
        near = np.nan_to_num(p[:, :1])
        q_vert = wl.mix_q(np.repeat(near, VSD, 1), wl.make_head_probs(B, VSD, V, vb, ve, seed), 0.6)
        q_horiz = wl.mix_q(np.repeat(near, K, 1), wl.make_head_probs(B, K, V, vb, ve, seed + 1), 0.6)
        u_pool = wl.draw_pool_uniforms(B, NQ, seed)
        uu = wl.draw_tree_uniforms(B, N, seed)
        cache.put(q_vert, position)
        want_q, _ = sp.pool_build(q_horiz, cache, position)
        ora_row, margin = sp.pool_sample(want_q, u_pool, vb, ve)
        ora_tok = sp.node_tokens(ora_row, node_q)
        ora = oracle.tree_accept(logits, want_q, ora_tok, node_q, child_begin, uu["u_accept"], uu["u_resample"], vb, ve,
                                 s, 1.0, top_k, max_depth=K)
        hawk.spec_cache_put(to_dev(q_vert), to_dev(position), rows, tags, IW)
        pool_q, _ = hawk.pool_build(to_dev(q_horiz), rows, tags, to_dev(position), IW, VSD, with_source=False)
        node_token = hawk.pool_sample(pool_q, to_dev(u_pool), to_dev(node_q), vb, ve)
        alen, otok, path = hawk.tree_accept(to_dev(logits), pool_q, node_token, to_dev(node_q), to_dev(child_begin),
                                            to_dev(uu["u_accept"]), to_dev(uu["u_resample"]), vb, ve, s, 1.0, top_k,
                                            max_depth=K)
        torch.cuda.synchronize()
        assert np.array_equal(pool_q.cpu().numpy(), want_q)
        alen, otok, path = alen.cpu().numpy(), otok.cpu().numpy(), path.cpu().numpy()
        tok_exempt = (margin[:, node_q] < TOL).any(axis=1)
        for b in range(B):
            if tok_exempt[b] or (ora["accept_margin"][b] < TOL).any():
                continue
            assert np.array_equal(node_token[b].cpu().numpy(), ora_tok[b])
            assert alen[b] == ora["accept_len"][b] and np.array_equal(path[b], ora["path"][b])
            if ora["resample_margin"][b] >= TOL:
                assert otok[b] == ora["token"][b]
        lens.append(ora["accept_len"].copy())
        position = (position + ora["accept_len"] + 1).astype(np.int32)      # the oracle's verdict drives both sides
    lens = np.concatenate(lens)
    assert lens.max() >= 1 and lens.min() == 0      # the walk both advanced and stopped at the root


def test_argument_errors():
    import paper_2510_25739_b200 as hawk
    from paper_2510_25739_b200 import binding
    lib = hawk.load_library()
    assert hawk.spec_cache_slots(0, 2) == 0 and hawk.spec_cache_slots(4, 0) == 0
    assert hawk.spec_cache_slot(4, 2, -1, 1) == -1 and hawk.spec_cache_slot(4, 2, 0, 3) == -1
    B, IW, VSD, K, V = 1, 4, 2, 2, 64
    rows, tags = hawk.spec_cache_new(B, IW, VSD, V)
    qv = to_dev(wl.make_head_probs(B, VSD, V, 0, V, 1))
    qh = to_dev(wl.make_head_probs(B, K, V, 0, V, 2))
    pos = to_dev(np.zeros(B, np.int32))
    P = binding._ptr
    st = binding._stream()
    assert lib.hawk_spec_cache_put(None, P(pos), P(rows), P(tags), B, IW, VSD, V, st) == 1       # NULL
    assert lib.hawk_spec_cache_put(P(qv), P(pos), P(rows), P(tags), B, 0, VSD, V, st) == 2       # SHAPE
    assert lib.hawk_spec_cache_put(P(qv), P(pos), P(rows), P(tags), B, IW, 9, V, st) == 4        # UNSUPPORTED
    assert lib.hawk_spec_cache_put(P(qv), P(pos), P(rows), P(tags), 0, IW, VSD, V, st) == 0      # nothing to do
    assert lib.hawk_spec_cache_clear(None, B, IW, VSD, st) == 1
    pool = torch.empty((B, K * (1 + VSD), V), dtype=torch.float32, device="cuda")
    assert lib.hawk_pool_build(P(qh), P(rows), P(tags), P(pos), None, None, B, K, IW, VSD, V, st) == 1
    assert lib.hawk_pool_build(P(qh), P(rows), P(tags), P(pos), P(pool), None, B, K, IW, VSD, 0, st) == 2
    assert lib.hawk_pool_build(P(qh), P(rows), P(tags), P(pos), P(pool), None, B, 0, IW, VSD, V, st) == 0
    NQ, N = K * (1 + VSD), 3
    u = to_dev(np.zeros((B, NQ), np.float32))
    nq = to_dev(np.zeros(N, np.int32))
    out = torch.empty((B, N), dtype=torch.int32, device="cuda")
    ws = torch.empty(64, dtype=torch.uint8, device="cuda")
    assert hawk.pool_sample_workspace_bytes(B, NQ) == 4 * B * NQ
    assert lib.hawk_pool_sample(P(pool), P(u), P(nq), P(out), B, NQ, N, V, 0, V, P(ws), 8, None, st) == 5   # WORKSPACE
    assert lib.hawk_pool_sample(P(pool), P(u), P(nq), P(out), B, NQ, N, V, 8, 8, P(ws), 64, None, st) == 2  # SHAPE
    assert lib.hawk_pool_sample(P(pool), P(u), None, P(out), B, NQ, N, V, 0, V, P(ws), 64, None, st) == 1   # NULL
    big = 40000
    assert lib.hawk_pool_sample(P(pool), P(u), P(nq), P(out), B, NQ, N, big, 0, big, P(ws), 64, None, st) == 4
    torch.cuda.synchronize()
