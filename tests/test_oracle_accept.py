"""Pins of the oracle's target distribution, acceptance rule and residual resampling.

Sources of truth: the speculative sampling rule (Sec. 3), first-rejection resampling from
norm(max(0, p - q)) (Sec. 4.2, Eq. "recur"), the acceptance probability
alpha = 1 - sum(p - min(q, p)) and the distribution-preservation identity (App. A).
"""
from pathlib import Path

import numpy as np
import pytest
from scipy.special import softmax
from scipy.stats import chi2

import oracle

GOLDEN = Path(__file__).parent / "golden" / "accept_worked_examples.txt"


def _stack(lc, lu):
    """[rows,V] conditional and unconditional rows of ONE sequence -> logits [2,rows,V]."""
    return np.stack([np.atleast_2d(lc), np.atleast_2d(lu)]).astype(np.float32)


def _accept_one(p_logits, q, draft, u_acc, u_res, **kw):
    V = len(p_logits)
    lg = _stack(p_logits, p_logits)
    return oracle.cfg_accept(lg, np.asarray(q, np.float32).reshape(1, 1, V),
                             np.array([[draft]], np.int32), np.array([[u_acc]], np.float32),
                             np.array([[u_res, 0.5]], np.float32), 0, V, 1.0, 1.0, 0, **kw)


# ---------------------------------------------------------------- target distribution
def test_guidance_scale_one_and_zero_select_a_stream():
    rng = np.random.default_rng(0)
    lc, lu = rng.standard_normal(50).astype(np.float32), rng.standard_normal(50).astype(np.float32)
    p1, _ = oracle.target_probs(lc, lu, 0, 50, 1.0, 1.0, 0)
    p0, _ = oracle.target_probs(lc, lu, 0, 50, 0.0, 1.0, 0)
    np.testing.assert_allclose(p1, softmax(lc.astype(np.float64)), rtol=2e-6)   # fp32 combine
    np.testing.assert_allclose(p0, softmax(lu.astype(np.float64)), rtol=1e-13)  # exact: 0*d + lu


def test_guidance_extrapolates_away_from_unconditional():
    lc = np.array([1.0, 0.0, -1.0], np.float32)
    lu = np.array([0.0, 0.0, 0.0], np.float32)
    p, _ = oracle.target_probs(lc, lu, 0, 3, 3.0, 1.0, 0)
    np.testing.assert_allclose(p, softmax(np.array([3.0, 0.0, -3.0])), rtol=1e-13)
    lu2 = np.array([0.5, 0.25, -2.0], np.float32)                 # all values exact in fp32
    p2, _ = oracle.target_probs(lc, lu2, 0, 3, 2.0, 1.0, 0)
    np.testing.assert_allclose(p2, softmax(np.array([1.5, -0.25, 0.0])), rtol=1e-13)


def test_temperature_divides_logits():
    lc = np.array([2.0, 1.0, 0.0, -4.0], np.float32)
    p, _ = oracle.target_probs(lc, lc, 0, 4, 1.0, 0.5, 0)
    np.testing.assert_allclose(p, softmax(np.array([4.0, 2.0, 0.0, -8.0])), rtol=1e-13)
    # scaling logits and temperature by the same power of two changes nothing at all
    pa, _ = oracle.target_probs(lc, lc, 0, 4, 1.0, 1.0, 0)
    pb, _ = oracle.target_probs(4 * lc, 4 * lc, 0, 4, 1.0, 4.0, 0)
    np.testing.assert_array_equal(pa, pb)


@pytest.mark.parametrize("V,k", [(64, 1), (64, 5), (64, 63), (1000, 200), (16384, 2000)])
def test_top_k_keeps_exactly_the_k_largest(V, k):
    rng = np.random.default_rng(V + k)
    lc, lu = rng.standard_normal(V).astype(np.float32), rng.standard_normal(V).astype(np.float32)
    p, _ = oracle.target_probs(lc, lu, 0, V, 2.5, 0.8, k)
    pfull, _ = oracle.target_probs(lc, lu, 0, V, 2.5, 0.8, 0)
    assert (p > 0).sum() == k                                    # continuous draws: no ties
    tau = np.partition(pfull, V - k)[V - k]                      # k-th largest by a library routine
    keep = pfull >= tau
    np.testing.assert_array_equal(p > 0, keep)
    np.testing.assert_allclose(p[keep], pfull[keep] / pfull[keep].sum(), rtol=1e-12)
    assert abs(p.sum() - 1) < 1e-12


def test_top_k_special_cases_and_ties():
    lc = np.array([0.0, 3.0, 1.0, 3.0, -1.0, 1.0], np.float32)
    for k in (0, -1, 6, 100):                                    # no filter
        p, _ = oracle.target_probs(lc, lc, 0, 6, 1.0, 1.0, k)
        np.testing.assert_allclose(p, softmax(lc.astype(np.float64)), rtol=1e-13)
    p, _ = oracle.target_probs(lc, lc, 0, 6, 1.0, 1.0, 1)        # tie at the top: both kept
    np.testing.assert_allclose(p, [0, .5, 0, .5, 0, 0], atol=1e-15)
    p, _ = oracle.target_probs(lc, lc, 0, 6, 1.0, 1.0, 3)        # threshold value 1.0 is tied: 4 kept
    assert (p > 0).tolist() == [False, True, True, True, False, True]
    one = np.array([0.0, 1.0, 5.0, 2.0], np.float32)
    p, _ = oracle.target_probs(one, one, 0, 4, 1.0, 1.0, 1)
    np.testing.assert_array_equal(p, [0, 0, 1, 0])


def test_masked_and_invalid_ids():
    lc = np.array([9.0, 1.0, -np.inf, 2.0, 0.0, 9.0], np.float32)
    lu = np.array([9.0, 1.0, 0.0, -np.inf, 0.0, 9.0], np.float32)
    p, flags = oracle.target_probs(lc, lu, 1, 5, 2.0, 1.0, 0)     # ids 0 and 5 outside the range
    assert flags == 0
    np.testing.assert_allclose(p, [0, np.e / (np.e + 1), 0, 0, 1 / (np.e + 1), 0], rtol=1e-13)
    lc[1] = np.nan
    p, flags = oracle.target_probs(lc, lu, 1, 5, 2.0, 1.0, 0)
    assert flags == oracle.FLAG_NONFINITE
    np.testing.assert_array_equal(p, [0, 0, 0, 0, 1, 0])
    # top-k counts finite entries only: k=2 of the 2 finite ones is "no filter"
    lc[1] = 1.0
    p2, _ = oracle.target_probs(lc, lu, 1, 5, 2.0, 1.0, 2)
    assert (p2 > 0).sum() == 2


# ---------------------------------------------------------------- worked examples (golden)
def _golden_cases():
    P = {"A": [1 / 2, 1 / 4, 1 / 8, 1 / 8], "B": [2 / 5, 3 / 10, 1 / 5, 1 / 10]}
    Q = {"A": [1 / 4, 1 / 2, 1 / 8, 1 / 8], "B": [1 / 10, 1 / 5, 3 / 10, 2 / 5]}
    for line in GOLDEN.read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        case, draft, ua, ur, alen, tok = line.split()
        yield P[case], Q[case], int(draft), float(ua), float(ur), int(alen), int(tok)


def test_hand_computed_examples():
    n = 0
    for p, q, draft, ua, ur, alen, tok in _golden_cases():
        out = _accept_one(np.log(np.array(p)), q, draft, ua, ur)
        assert (out["accept_len"][0], out["token"][0]) == (alen, tok), (p, q, draft, ua, ur)
        n += 1
    assert n == 12


def test_residual_and_acceptance_probability_of_worked_examples():
    p = np.array([2 / 5, 3 / 10, 1 / 5, 1 / 10]); q = np.array([1 / 10, 1 / 5, 3 / 10, 2 / 5], np.float32)
    r, total = oracle.residual(p, q, 0, 4)
    np.testing.assert_allclose(r, [0.3, 0.1, 0, 0], atol=1e-7)
    assert abs(total - 0.4) < 1e-7
    assert abs((1 - total) - np.minimum(p, q).sum()) < 1e-7      # alpha = 1 - residual mass


# ---------------------------------------------------------------- acceptance rule
def test_q_equal_p_accepts_every_draft_for_any_uniform():
    rng = np.random.default_rng(1)
    B, K, V = 16, 6, 64
    lg = rng.standard_normal((2 * B, K, V)).astype(np.float32)
    p, _ = oracle.target_probs_rows(lg, 0, V, 3.0, 1.0, 20)
    q = p.astype(np.float32)
    draft = np.stack([[rng.choice(V, p=p[b, i]) for i in range(K)] for b in range(B)]).astype(np.int32)
    for u in (0.0, 0.5, np.nextafter(np.float32(1), np.float32(0))):
        # q is p rounded to fp32: u*q < p needs u < 1 and q(x) <= p(x)(1+2^-24); use u just under 1
        # only where rounding went down, otherwise the strict test is decided by the rounding
        ua = np.full((B, K), u, np.float32)
        out = oracle.cfg_accept(lg, q, draft, ua, np.zeros((B, K + 1), np.float32), 0, V, 3.0, 1.0, 20)
        if u < 0.9:
            assert (out["accept_len"] == K).all() and (out["token"] == -1).all()
        else:
            assert (out["accept_margin"][out["accept_len"] < K] < 1e-6).all()


def test_disjoint_support_accepts_nothing_and_resamples_from_p():
    rng = np.random.default_rng(2)
    B, K, V = 32, 4, 64
    lg = rng.standard_normal((2 * B, K, V)).astype(np.float32)
    lg[:, :, 1::2] = -np.inf                                     # target lives on even ids
    q = np.zeros((B, K, V), np.float32)
    q[:, :, 1::2] = softmax(rng.standard_normal((B, K, V // 2)), axis=-1)
    draft = (2 * rng.integers(0, V // 2, (B, K)) + 1).astype(np.int32)
    ures = rng.random((B, K + 1)).astype(np.float32)
    out = oracle.cfg_accept(lg, q, draft, np.zeros((B, K), np.float32), ures, 0, V, 2.0, 1.0, 0)
    assert (out["accept_len"] == 0).all()
    p, _ = oracle.target_probs_rows(lg, 0, V, 2.0, 1.0, 0)
    for b in range(B):
        r, total = oracle.residual(p[b, 0], q[b, 0], 0, V)
        np.testing.assert_allclose(r, p[b, 0], rtol=1e-15)
        assert abs(total - 1) < 1e-12
        cdf = np.cumsum(p[b, 0])
        assert out["token"][b] == int(np.argmax(cdf > float(ures[b, 0])))
        assert out["token"][b] % 2 == 0


def test_zero_probability_corner_cases():
    logp = np.log(np.array([0.5, 0.5, 1e-30, 1e-30]))
    logp[2:] = -np.inf                                            # p = [.5,.5,0,0]
    # p(x)=0 < q(x): always rejected, even at u = 0
    assert _accept_one(logp, [0.25, 0.25, 0.5, 0.0], 2, 0.0, 0.3)["accept_len"][0] == 0
    # q(x)=0 < p(x): always accepted
    assert _accept_one(logp, [0.0, 0.5, 0.5, 0.0], 0, 0.999, 0.3)["accept_len"][0] == 1
    # 0/0: rejected
    assert _accept_one(logp, [0.5, 0.5, 0.0, 0.0], 3, 0.0, 0.3)["accept_len"][0] == 0
    # residual with no mass (q == p exactly) falls back to p with the same uniform
    out = _accept_one(logp, [0.5, 0.5, 0.0, 0.0], 3, 0.0, 0.75)
    assert out["token"][0] == 1
    out = _accept_one(logp, [0.5, 0.5, 0.0, 0.0], 3, 0.0, 0.25)
    assert out["token"][0] == 0


def test_inverse_cdf_end_points():
    logp = np.log(np.array([0.1, 0.2, 0.3, 0.4]))
    q = [0.1, 0.0, 0.9, 0.0]            # residual = [0, .2, 0, .4]: ids 1 and 3 only
    assert _accept_one(logp, q, 2, 0.9, 0.0)["token"][0] == 1
    assert _accept_one(logp, q, 2, 0.9, np.nextafter(np.float32(1), np.float32(0)))["token"][0] == 3
    assert _accept_one(logp, q, 2, 0.9, 0.3333)["token"][0] == 1
    assert _accept_one(logp, q, 2, 0.9, 0.3334)["token"][0] == 3
    q1 = [0.1, 0.2, 0.7, 0.0]           # one-hot residual at id 3
    for u in (0.0, 0.5, 0.999):
        assert _accept_one(logp, q1, 2, 0.9, u)["token"][0] == 3


def test_chain_stops_at_first_rejection_and_bonus_row():
    V, K = 8, 3
    rng = np.random.default_rng(5)
    lg = rng.standard_normal((2, K + 1, V)).astype(np.float32)
    p, _ = oracle.target_probs_rows(lg, 0, V, 2.0, 1.0, 0)
    q = p[:, :K].astype(np.float32)
    draft = np.array([[1, 2, 3]], np.int32)
    ures = np.array([[0.1, 0.2, 0.3, 0.6]], np.float32)
    # all accepted, bonus row sampled from p of row K with u_resample[K]
    out = oracle.cfg_accept(lg, q, draft, np.full((1, K), 0.5, np.float32), ures, 0, V, 2.0, 1.0, 0,
                            has_bonus_row=True)
    assert out["accept_len"][0] == K
    assert out["token"][0] == int(np.argmax(np.cumsum(p[0, K]) > 0.6))
    # force a rejection at position 1 by giving the draft there no target mass
    lg2 = lg.copy(); lg2[:, 1, 2] = -np.inf
    q2 = q.copy(); q2[0, 1] = 0; q2[0, 1, 2] = 1.0
    out = oracle.cfg_accept(lg2, q2, draft, np.full((1, K), 0.5, np.float32), ures, 0, V, 2.0, 1.0, 0,
                            has_bonus_row=True)
    p2, _ = oracle.target_probs_rows(lg2, 0, V, 2.0, 1.0, 0)
    assert out["accept_len"][0] == 1
    assert out["token"][0] == int(np.argmax(np.cumsum(p2[0, 1]) > 0.2))   # residual == p there
    assert np.isnan(out["ratio"][0, 2])                                   # position 2 never examined


def test_out_of_range_draft_is_clamped_and_flagged():
    logp = np.log(np.array([0.25, 0.25, 0.25, 0.25]))
    out = _accept_one(logp, [0.25] * 4, 7, 0.5, 0.5)
    assert out["flags"] & oracle.FLAG_BAD_DRAFT


# ---------------------------------------------------------------- statistics
def _dist_pair(rng, V, top_k=0):
    lc, lu = rng.standard_normal(V).astype(np.float32), rng.standard_normal(V).astype(np.float32)
    p, _ = oracle.target_probs(lc, lu, 0, V, 2.0, 1.0, top_k)
    q = (0.6 * p + 0.4 * softmax(rng.standard_normal(V))).astype(np.float32)
    return lc, lu, p, q


def test_distribution_preservation_identity_exact():
    rng = np.random.default_rng(21)
    for top_k in (0, 10):
        _, _, p, q = _dist_pair(rng, 64, top_k)
        qd = q.astype(np.float64)
        r, total = oracle.residual(p, q, 0, 64)
        alpha = np.minimum(p, qd).sum()
        assert abs((1 - alpha) - total) < 1e-12 + abs(1 - qd.sum())
        accept_prob = np.where(qd > 0, np.minimum(1.0, p / np.where(qd > 0, qd, 1)), 0)
        emitted = qd * accept_prob + (1 - (qd * accept_prob).sum()) * r / total
        np.testing.assert_allclose(emitted, p, atol=2e-8)        # q carries fp32 rounding


def test_emitted_token_follows_p_chi_square():
    rng = np.random.default_rng(22)
    V, N = 64, 100_000
    lc, lu, p, q = _dist_pair(rng, V)
    lg = np.empty((2 * N, 1, V), np.float32); lg[:N, 0] = lc; lg[N:, 0] = lu
    qq = np.broadcast_to(q, (N, 1, V)).copy()
    cdf = np.cumsum(q.astype(np.float64)); cdf /= cdf[-1]
    draft = np.searchsorted(cdf, rng.random(N), side="right").clip(0, V - 1).astype(np.int32)[:, None]
    out = oracle.cfg_accept(lg, qq, draft, rng.random((N, 1), dtype=np.float32),
                            rng.random((N, 2), dtype=np.float32), 0, V, 2.0, 1.0, 0, diagnostics=False)
    emitted = np.where(out["accept_len"] == 1, draft[:, 0], out["token"])
    counts = np.bincount(emitted, minlength=V)
    stat = ((counts - N * p) ** 2 / (N * p)).sum()
    assert stat < chi2.ppf(0.999, V - 1)                          # 103.44 for 63 degrees of freedom
    # acceptance rate equals sum(min(p, q)) within 4 binomial standard deviations
    beta = np.minimum(p, q).sum()
    rate = (out["accept_len"] == 1).mean()
    assert abs(rate - beta) < 4 * np.sqrt(beta * (1 - beta) / N)
    # a wrong rule would not pass: the drafts alone (distributed as q) fail the same test
    cq = np.bincount(draft[:, 0], minlength=V)
    assert ((cq - N * p) ** 2 / (N * p)).sum() > chi2.ppf(0.999, V - 1)


def test_expected_accept_length_of_a_chain():
    rng = np.random.default_rng(23)
    V, K, N = 32, 4, 40_000
    rows = [_dist_pair(rng, V) for _ in range(K)]
    beta = np.array([np.minimum(p, q).sum() for _, _, p, q in rows])
    lg = np.empty((2 * N, K, V), np.float32)
    qq = np.empty((N, K, V), np.float32)
    draft = np.empty((N, K), np.int32)
    for i, (lc, lu, p, q) in enumerate(rows):
        lg[:N, i] = lc; lg[N:, i] = lu; qq[:, i] = q
        cdf = np.cumsum(q.astype(np.float64)); cdf /= cdf[-1]
        draft[:, i] = np.searchsorted(cdf, rng.random(N), side="right").clip(0, V - 1)
    out = oracle.cfg_accept(lg, qq, draft, rng.random((N, K), dtype=np.float32),
                            rng.random((N, K + 1), dtype=np.float32), 0, V, 2.0, 1.0, 0,
                            diagnostics=False)
    expect = np.cumprod(beta).sum()
    var_bound = K * K / 4
    assert abs(out["accept_len"].mean() - expect) < 4 * np.sqrt(var_bound / N)
    # P(accept_len >= j) = prod_{i<j} beta_i
    for j in range(1, K + 1):
        pj = np.prod(beta[:j])
        assert abs((out["accept_len"] >= j).mean() - pj) < 4 * np.sqrt(pj * (1 - pj) / N) + 1e-9
