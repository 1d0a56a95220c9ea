"""hawk_cfg_accept_noalloc against hawk_cfg_accept, through the C ABI.

The no-allocation entry point serves callers that own no spare device memory when they need a
verdict (a decode loop inside an engine that reserved the whole GPU up front; a plug-in that only
receives input and output buffers).  It must give exactly what the workspace-taking call gives: same
kernels, only the verdict scratch lives in the library's built-in array.  Two different steps are run
back to back, so that the second one meets the array still holding the first one's verdicts.
This file sorts last on purpose: a run that stops at the first failure has already run the rest.
"""
import numpy as np
import pytest
import torch

from paper_2510_25739_b200 import workloads as wl
from tests._util import to_dev

pytestmark = pytest.mark.gpu


def _step_inputs(cfg, seed, bonus):
    logits = wl.make_logits(cfg, seed, has_bonus_row=bonus)
    q = wl.random_probs(cfg, seed).astype(np.float32)
    u = wl.draw_uniforms(cfg, seed)
    return [to_dev(a) for a in (logits, q, wl.draw_drafts(q, seed), u["u_accept"], u["u_resample"])]


def test_matches_the_workspace_call_twice_in_a_row():
    import paper_2510_25739_b200 as hawk
    assert hawk.cfg_accept_noalloc_max_rows() >= 64 * 9
    steps = [
        (wl.config(2, B=8, K=5), 4100, False),                                     # 16384 ids, top-k 2000
        (wl.config(4, B=3, K=6, V=65536, v_begin=4, v_end=8196), 4200, True),      # offset range, bonus row
    ]
    for cfg, seed, bonus in steps:
        args = _step_inputs(cfg, seed, bonus)
        params = (cfg.v_begin, cfg.v_end, cfg.cfg_scale, cfg.temperature, cfg.top_k)
        want_len, want_tok = hawk.cfg_accept(*args, *params, has_bonus_row=bonus)
        got_len = torch.full((cfg.B,), -7, dtype=torch.int32, device="cuda")
        got_tok = torch.full((cfg.B,), -7, dtype=torch.int32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        hawk.cfg_accept_noalloc(*args, *params, got_len, got_tok, has_bonus_row=bonus, dev_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        # integer results: bit-exact, as everywhere else in the accept tests
        assert torch.equal(got_len, want_len) and torch.equal(got_tok, want_tok)
        assert int(got_len.min()) >= 0 and int(got_len.max()) <= cfg.K


def test_many_rows_twice_with_different_inputs():
    """A step of 64 sequences x 8 drafts: more than 1.5 rows per SM, so the call first marks every verdict slot of
    the built-in array unknown and rows behind a rejection return early.  The second step has other inputs and
    meets the array still holding the first step's verdicts; both must equal the workspace-taking call."""
    import paper_2510_25739_b200 as hawk
    import oracle
    cfg = wl.config(5, top_k=0, q_alpha=0.6)
    assert cfg.B * cfg.K > 222
    for seed, bonus in ((4300, False), (4301, True)):
        args = _step_inputs(cfg, seed, bonus)
        # drafts that are partly accepted: q mixed with the target distribution (input recipe only; the expected
        # values below come from the workspace-taking call, not from the oracle)
        p, _ = oracle.target_probs_rows(args[0].cpu().numpy(), cfg.v_begin, cfg.v_end, cfg.cfg_scale, cfg.temperature,
                                        cfg.top_k)
        q = wl.make_q(cfg, seed, np.nan_to_num(p[:, :cfg.K]))
        args[1], args[2] = to_dev(q), to_dev(wl.draw_drafts(q, seed))
        params = (cfg.v_begin, cfg.v_end, cfg.cfg_scale, cfg.temperature, cfg.top_k)
        want_len, want_tok = hawk.cfg_accept(*args, *params, has_bonus_row=bonus)
        got_len = torch.full((cfg.B,), -7, dtype=torch.int32, device="cuda")
        got_tok = torch.full((cfg.B,), -7, dtype=torch.int32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        hawk.cfg_accept_noalloc(*args, *params, got_len, got_tok, has_bonus_row=bonus, dev_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(got_len, want_len) and torch.equal(got_tok, want_tok)
        assert 0 < float(got_len.float().mean()) < cfg.K     # the step has both accepted and rejected drafts


def test_step_larger_than_the_builtin_array_is_refused():
    import paper_2510_25739_b200 as hawk
    from paper_2510_25739_b200.binding import HawkError
    K, V = 16, 64
    B = hawk.cfg_accept_noalloc_max_rows() // (K + 1) + 1
    dev = "cuda"
    logits = torch.zeros((2 * B, K, V), device=dev)
    q = torch.full((B, K, V), 1.0 / V, device=dev)
    draft = torch.zeros((B, K), dtype=torch.int32, device=dev)
    ua, ur = torch.zeros((B, K), device=dev), torch.zeros((B, K + 1), device=dev)
    out_len = torch.full((B,), -7, dtype=torch.int32, device=dev)
    out_tok = torch.full((B,), -7, dtype=torch.int32, device=dev)
    with pytest.raises(HawkError) as err:
        hawk.cfg_accept_noalloc(logits, q, draft, ua, ur, 0, V, 1.0, 1.0, 0, out_len, out_tok)
    assert err.value.code == 5                       # workspace: the built-in array is too small
    torch.cuda.synchronize()
    assert (out_len == -7).all() and (out_tok == -7).all()   # nothing ran
