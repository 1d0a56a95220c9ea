"""GPU parity of hawk_tree_accept (candidate tree, recursive residual) against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_25739_b200 import workloads as wl
from tests._util import to_dev

pytestmark = pytest.mark.gpu
TOL = 1e-5


def _compare(got_len, got_tok, got_path, ora):
    """Bit-exact accepted length, path and token; a sequence is exempt when a candidate it examined
    lies within TOL of its acceptance threshold, its token when the draw lies within TOL of a CDF boundary."""
    bad, exempt_acc, exempt_res, checked = [], 0, 0, 0
    for b in range(len(got_len)):
        if (ora["accept_margin"][b] < TOL).any():
            exempt_acc += 1
            continue
        if got_len[b] != ora["accept_len"][b] or (got_path[b] != ora["path"][b]).any():
            bad.append((b, "path", got_path[b].tolist(), ora["path"][b].tolist()))
            continue
        if ora["resample_margin"][b] < TOL:
            exempt_res += 1
            continue
        checked += 1
        if got_tok[b] != ora["token"][b]:
            bad.append((b, "tok", int(got_tok[b]), int(ora["token"][b])))
    return dict(bad=bad, exempt_accept=exempt_acc, exempt_resample=exempt_res, checked=checked)


def _case(B, V, vb, ve, top_k, branching, seed, alpha=0.7, cfg_scale=3.0, expect_flags=0, mutate=None):
    import paper_2510_25739_b200 as hawk
    tree = wl.make_tree(branching)
    N, NQ = tree["N"], tree["NQ"]
    cfg = wl.config(2, B=B, K=N, V=V, v_begin=vb, v_end=ve, top_k=top_k, cfg_scale=cfg_scale, H=4, H_kv=4)
    logits = wl.make_logits(cfg, seed)                                  # [2B, N, V]
    p, _ = oracle.target_probs_rows(logits, vb, ve, cfg_scale, 1.0, top_k)
    first_of_depth = [int(np.argmax(tree["node_depth"] == d)) for d in range(len(branching))]
    r = wl.random_probs(wl.config(2, B=B, K=NQ, V=V, v_begin=vb, v_end=ve), seed)      # [B, NQ, V]
    width = max(branching)
    p_for_q = np.stack([np.nan_to_num(p[:, first_of_depth[j // width]]) for j in range(NQ)], axis=1)
    q = wl.mix_q(p_for_q, r, alpha)
    tok = wl.draw_tree_tokens(q, tree, seed)
    u = wl.draw_tree_uniforms(B, N, seed)
    child_begin, node_q = tree["child_begin"].copy(), tree["node_q"].copy()
    if mutate:
        mutate(child_begin, node_q, tok)
    ora = oracle.tree_accept(logits, q, tok, node_q, child_begin, u["u_accept"], u["u_resample"], vb, ve,
                             cfg_scale, 1.0, top_k, max_depth=len(branching)) if not mutate else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    alen, otok, path = hawk.tree_accept(to_dev(logits), to_dev(q), to_dev(tok), to_dev(node_q), to_dev(child_begin),
                                        to_dev(u["u_accept"]), to_dev(u["u_resample"]), vb, ve, cfg_scale, 1.0,
                                        top_k, max_depth=len(branching), dev_status=status)
    torch.cuda.synchronize()
    got = alen.cpu().numpy(), otok.cpu().numpy(), path.cpu().numpy()
    if mutate:
        return got, int(status.item())
    assert int(status.item()) == expect_flags
    res = _compare(*got, ora)
    assert not res["bad"], res["bad"][:5]
    return res, ora


@pytest.mark.parametrize("B,V,vb,ve,top_k,branching", [
    (4, 64, 0, 64, 0, (2,)),
    (6, 1000, 3, 999, 100, (3, 2)),
    (5, 4096, 0, 4096, 500, (2, 2, 2)),
    (8, 16384, 0, 16384, 2000, (3, 2, 2)),
    (3, 65536, 4, 8196, 2000, (4, 1, 3)),
    (6, 20000, 0, 20000, 0, (2, 2)),
    (16, 16384, 0, 16384, 2000, (1, 1, 1, 1, 1)),       # a chain
    (24, 4096, 0, 4096, 300, (3, 2, 2)),                # 528 rows: more than 1.5 waves, unreachable nodes do no work
    (40, 1000, 4, 996, 50, (2, 2, 2)),                  # 600 narrow rows
])
def test_matches_oracle(B, V, vb, ve, top_k, branching):
    res, ora = _case(B, V, vb, ve, top_k, branching, seed=300 + V + len(branching))
    # without top-k every id carries ~1/V of the mass, the same order as the exemption band around a
    # CDF boundary: there the token of most sequences is exempt and the test checks lengths and paths
    assert res["exempt_accept"] <= max(1, B // 4)
    assert res["exempt_resample"] <= (B if top_k == 0 else max(1, B // 4))


@pytest.mark.parametrize("alpha", [0.0, 0.5, 0.95])
def test_accept_lengths_spread_with_draft_quality(alpha):
    res, ora = _case(32, 16384, 0, 16384, 2000, (3, 2, 2), seed=900 + int(alpha * 100), alpha=alpha)
    if alpha >= 0.9:
        assert ora["accept_len"].mean() > 1.0            # good drafts: the walk goes deep
    print(f"alpha {alpha}: mean accept_len {ora['accept_len'].mean():.2f}, checked {res['checked']}")


def test_second_head_rescues_a_rejected_level():
    """With the first head useless (disjoint from the target) and the second one good, every sequence
    still advances: the point of drawing the candidates of a level from different heads."""
    import paper_2510_25739_b200 as hawk
    B, V = 8, 4096
    tree = wl.make_tree((2,))
    cfg = wl.config(2, B=B, K=3, V=V, v_begin=0, v_end=V, top_k=0, cfg_scale=1.0, H=4, H_kv=4)
    logits = wl.mask_odd_ids(wl.make_logits(cfg, 5), cfg)               # target lives on even ids
    p, _ = oracle.target_probs_rows(logits, 0, V, 1.0, 1.0, 0)
    q = np.stack([wl.random_probs(wl.config(2, B=B, K=1, V=V, v_begin=0, v_end=V), 5, only_odd=True)[:, 0],
                  p[:, 0]], axis=1).astype(np.float32)                  # head 0 on odd ids, head 1 = target
    tok = wl.draw_tree_tokens(q, tree, 5)
    u = wl.draw_tree_uniforms(B, 3, 5)
    alen, otok, path = hawk.tree_accept(to_dev(logits), to_dev(q), to_dev(tok), to_dev(tree["node_q"]),
                                        to_dev(tree["child_begin"]), to_dev(u["u_accept"]), to_dev(u["u_resample"]),
                                        0, V, 1.0, 1.0, 0, max_depth=1)
    ora = oracle.tree_accept(logits, q, tok, tree["node_q"], tree["child_begin"], u["u_accept"], u["u_resample"],
                             0, V, 1.0, 1.0, 0, max_depth=1)
    near = (ora["accept_margin"] < TOL).any(axis=1)
    assert (alen.cpu().numpy()[~near] == 1).all() and (path.cpu().numpy()[~near, 0] == 2).all()
    assert (ora["accept_len"][~near] == 1).all()


def test_malformed_tree_is_clamped_flagged_and_ends():
    from paper_2510_25739_b200 import binding

    def mutate(child_begin, node_q, tok):
        child_begin[0] = 0          # the root as its own child: clamped to node + 1
        node_q[2] = 99              # draft row out of range
    (alen, otok, path), status = _case(4, 1024, 0, 1024, 50, (2, 2), seed=77, mutate=mutate)
    assert status & binding.DEV_BAD_TREE
    assert ((alen >= 0) & (alen <= 2)).all()
