"""Pins of the oracle's training-side quantities (reverse KL, expected acceptance, alignment divergence,
group-relative advantage, sliding window scores, proportional draw of a window start) against library
routines, closed forms, invariants and brute force.  CPU only."""
import math

import numpy as np
import pytest
import scipy.special as sps
import scipy.stats as sst

import oracle


def _rand_case(rng, N, K, V, sigma=0.7):
    t = (rng.normal(size=(N, K, V)) * 2.0).astype(np.float32)
    d = (t + sigma * rng.normal(size=(N, K, V))).astype(np.float32)
    tok = rng.integers(0, V, size=(N, K)).astype(np.int32)
    return d, t, tok


# ------------------------------------------------------------------ reverse KL, expected acceptance, nabla


@pytest.mark.parametrize("T", [1.0, 0.6])
@pytest.mark.parametrize("V", [2, 19, 700])
def test_reverse_kl_and_expected_acceptance_match_scipy(T, V):
    rng = np.random.default_rng(V + int(10 * T))
    d, t, tok = _rand_case(rng, 4, 3, V)
    o = oracle.diagnostics(d, t, tok, temperature=T)
    P = sps.softmax(t.astype(np.float64) / T, axis=-1)
    Q = sps.softmax(d.astype(np.float64) / T, axis=-1)
    np.testing.assert_allclose(o["kl_rev"], sps.rel_entr(Q, P).sum(-1), rtol=1e-9, atol=1e-13)
    np.testing.assert_allclose(o["kl_rev_mean"], sps.rel_entr(Q, P).sum(-1).mean(-1), rtol=1e-9, atol=1e-13)
    tv = 0.5 * np.abs(P - Q).sum(-1)
    np.testing.assert_allclose(o["expected_accept"], 1.0 - tv, rtol=1e-11, atol=1e-13)        # App. B.1 identity
    lp = np.log(np.take_along_axis(P, tok[..., None].astype(np.int64), -1)[..., 0])
    lq = np.log(np.take_along_axis(Q, tok[..., None].astype(np.int64), -1)[..., 0])
    np.testing.assert_allclose(o["nabla"], np.exp(lp - lq) - (lp - lq) - 1.0, rtol=1e-7, atol=1e-12)
    # direction matters: the forward KL of the scoring pass is a different number
    fwd = oracle.score_windows(d, t, tok, mode=oracle.GREEDY, c=0.05, temperature=T)["kl"]
    assert not np.allclose(fwd, o["kl_rev"], rtol=1e-3)
    # Pinsker holds for either direction (App. B.1)
    assert np.all(tv <= np.sqrt(0.5 * o["kl_rev"]) + 1e-12) and np.all(tv <= np.sqrt(0.5 * fwd) + 1e-12)


def test_reverse_kl_closed_forms():
    # P = (1/4, 3/4), Q = (1/2, 1/2):  KL(Q||P) = 1/2 ln 2 + 1/2 ln(2/3);  sum min = 1/4 + 1/2
    t = np.array([[[0.0, math.log(3.0)]]], np.float32)
    d = np.array([[[0.0, 0.0]]], np.float32)
    o = oracle.diagnostics(d, t, np.array([[1]], np.int32))
    assert o["kl_rev"][0, 0] == pytest.approx(0.5 * math.log(2.0) + 0.5 * math.log(2.0 / 3.0), rel=1e-7)
    assert o["expected_accept"][0, 0] == pytest.approx(0.75, rel=1e-7)
    # token 1: d = ln(3/4) - ln(1/2) = ln 1.5 ; nabla = 1.5 - ln 1.5 - 1
    assert o["nabla"][0, 0] == pytest.approx(0.5 - math.log(1.5), rel=1e-6)
    # identical distributions: all three are exactly their neutral values
    o = oracle.diagnostics(t, t, np.array([[0]], np.int32))
    assert o["kl_rev"][0, 0] == 0.0 and o["nabla"][0, 0] == 0.0 and o["expected_accept"][0, 0] == pytest.approx(1.0, abs=1e-15)


def test_nabla_properties():
    rng = np.random.default_rng(5)
    d, t, tok = _rand_case(rng, 20, 4, 50, sigma=2.0)
    o = oracle.diagnostics(d, t, tok)
    assert np.all(o["nabla"] >= 0.0)                       # e^x - x - 1 >= 0
    s = oracle.score_windows(d, t, tok, mode=oracle.GREEDY, c=0.05)
    dlt = s["logp_tok"] - s["logq_tok"]
    np.testing.assert_allclose(o["nabla"], np.expm1(dlt) - dlt, rtol=1e-9, atol=1e-14)
    tok[0, 0] = 50                                          # not a vocabulary entry
    assert oracle.diagnostics(d, t, tok)["nabla"][0, 0] == np.inf


def test_masked_positions_and_window_mean():
    rng = np.random.default_rng(6)
    d, t, tok = _rand_case(rng, 5, 6, 40)
    vl = np.array([6, 0, 3, 1, 5], np.int32)
    o = oracle.diagnostics(d, t, tok, valid_len=vl)
    full = oracle.diagnostics(d, t, tok)
    for n, L in enumerate(vl):
        assert np.all(o["kl_rev"][n, L:] == 0) and np.all(o["nabla"][n, L:] == 0) and np.all(o["expected_accept"][n, L:] == 0)
        np.testing.assert_array_equal(o["kl_rev"][n, :L], full["kl_rev"][n, :L])
        assert o["kl_rev_mean"][n] == pytest.approx(full["kl_rev"][n, :L].mean() if L else 0.0, rel=1e-12)


# ------------------------------------------------------------------ group-relative advantage


def test_group_advantage_closed_forms_and_invariants():
    # rewards (0, 1): mu = 1/2, population sigma = 1/2
    a = oracle.group_advantage(np.array([0.0, 1.0]), 2, delta=0.25)
    np.testing.assert_allclose(a, [-0.5 / 0.75, 0.5 / 0.75], rtol=1e-15)
    # constant group: zero advantage (not NaN) thanks to delta; group of one: zero
    assert np.all(oracle.group_advantage(np.full(8, 3.0), 8, delta=1e-6) == 0.0)
    assert np.all(oracle.group_advantage(np.arange(5.0), 1, delta=1e-6) == 0.0)
    rng = np.random.default_rng(7)
    r = rng.random(64) * 5
    G, delta = 8, 1e-3
    a = oracle.group_advantage(r, G, delta=delta).reshape(-1, G)
    rg = r.reshape(-1, G)
    np.testing.assert_allclose(a, (rg - rg.mean(1, keepdims=True)) / (rg.std(1, keepdims=True) + delta), rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(a.mean(1), 0.0, atol=1e-14)                                       # centred per group
    np.testing.assert_allclose(a.std(1), rg.std(1) / (rg.std(1) + delta), rtol=1e-12)            # unit scale up to delta
    # invariant under shifting a group's rewards, and ranks within the group are kept
    np.testing.assert_allclose(oracle.group_advantage(r + 10.0, G, delta=delta), a.ravel(), rtol=1e-9, atol=1e-12)
    assert np.array_equal(np.argsort(a, 1), np.argsort(rg, 1))
    with pytest.raises(RuntimeError):
        oracle.group_advantage(np.zeros(10), 4)                                                  # 10 is not a multiple of 4


def test_group_advantage_of_the_reward_column_printed_in_the_paper():
    # App. D prints R_speedup for k = 1..7; a rollout group of 8 windows with k = 0..7 (gamma = 0.1247)
    k = np.arange(8.0)
    r = k / (k * 0.1247 + 1.0)
    a = oracle.group_advantage(r, 8, delta=0.0)
    assert np.all(np.diff(a) > 0) and a.mean() == pytest.approx(0.0, abs=1e-14) and a.std() == pytest.approx(1.0, rel=1e-12)


# ------------------------------------------------------------------ sliding window scores and the draw of a start


def test_sliding_scores_match_convolution_and_brute_force():
    rng = np.random.default_rng(8)
    for T, K in ((1, 1), (10, 10), (37, 10), (200, 7), (5, 8)):
        v = rng.random(T)
        s = oracle.sliding_scores(v, K)
        if T < K:
            assert s.size == 0
            continue
        assert s.shape == (T - K + 1,)
        np.testing.assert_allclose(s, np.convolve(v, np.ones(K) / K, mode="valid"), rtol=1e-12)
        np.testing.assert_allclose(s, [v[j:j + K].mean() for j in range(T - K + 1)], rtol=1e-13)
    # K = T: the single window is the mean of everything, as in the independent-window score
    v = rng.random(12)
    assert oracle.sliding_scores(v, 12)[0] == pytest.approx(v.mean(), rel=1e-14)


def test_sample_start_is_the_inverse_cdf():
    s = np.array([0.0, 1.0, 0.0, 3.0, 0.0])
    assert oracle.sample_start(s, 0.0) == 1                   # zero-weight starts are never drawn
    assert oracle.sample_start(s, 0.2499) == 1 and oracle.sample_start(s, 0.2501) == 3
    assert oracle.sample_start(s, 0.999999) == 3
    assert oracle.sample_start(np.zeros(4), 0.6) == 2         # no signal: uniform
    assert oracle.sample_start(np.zeros(0), 0.3) == -1
    rng = np.random.default_rng(9)
    w = rng.random(12)
    us = rng.random(40000)
    draws = np.array([oracle.sample_start(w, u) for u in us])
    np.testing.assert_array_equal(draws, np.searchsorted(np.cumsum(w), us * w.sum(), side="right"))
    counts = np.bincount(draws, minlength=12)
    assert sst.chisquare(counts, w / w.sum() * len(us)).pvalue > 1e-4   # drawn in proportion to the weights


def test_mixed_draw_reduces_to_its_two_branches_and_mixes_in_the_stated_proportion():
    # hard-window curriculum (App. A, training configuration): a share hard_frac of the starts comes from the
    # ADAW draw, the rest is uniform over the starts
    rng = np.random.default_rng(21)
    w = rng.random(9) ** 3
    n = len(w)
    us = rng.random((30000, 2))
    # hard_frac = 1: always the ADAW draw, whatever the coin; hard_frac = 0: always floor(u * n)
    for um, ud in us[:2000]:
        assert oracle.sample_start_mixed(w, 1.0, um, ud) == oracle.sample_start(w, ud)
        assert oracle.sample_start_mixed(w, 0.0, um, ud) == int(ud * n)
    # the coin is strict: u_mix == hard_frac takes the uniform branch, the next float below takes ADAW
    s = np.array([0.0, 0.0, 0.0, 5.0])
    assert oracle.sample_start_mixed(s, 0.4, 0.4, 0.1) == 0
    assert oracle.sample_start_mixed(s, 0.4, np.nextafter(0.4, 0.0), 0.1) == 3
    assert oracle.sample_start_mixed(np.zeros(0), 0.4, 0.1, 0.1) == -1
    assert oracle.sample_start_mixed(s, 0.4, 0.9, 0.999999) == 3          # uniform branch reaches the last start
    # branch by branch against numpy, then the mixture frequencies against hard_frac * w/sum(w) + (1 - hard_frac)/n
    for hf in (0.2, 0.4, 0.6):                                             # the three stages the paper lists
        draws = np.array([oracle.sample_start_mixed(w, hf, um, ud) for um, ud in us])
        adaw = np.searchsorted(np.cumsum(w), us[:, 1] * w.sum(), side="right")
        unif = np.floor(us[:, 1] * n).astype(int)
        np.testing.assert_array_equal(draws, np.where(us[:, 0] < hf, adaw, unif))
        expect = (hf * w / w.sum() + (1.0 - hf) / n) * len(us)
        assert sst.chisquare(np.bincount(draws, minlength=n), expect).pvalue > 1e-4
        # and it is NOT either pure branch: the pure-ADAW and pure-uniform frequencies are rejected
        assert sst.chisquare(np.bincount(draws, minlength=n), w / w.sum() * len(us)).pvalue < 1e-6
        assert sst.chisquare(np.bincount(draws, minlength=n), np.full(n, len(us) / n)).pvalue < 1e-6


# ------------------------------------------------------------------ reference-window log-probability (exact Delta)


def test_reference_logprob_matches_scipy_and_links_the_two_forms_of_delta():
    rng = np.random.default_rng(10)
    d, t, tok = _rand_case(rng, 6, 5, 300)
    vl = np.array([5, 3, 0, 1, 5, 4], np.int32)
    for T in (1.0, 0.7):
        r = oracle.reference_logprob(t, temperature=T, valid_len=vl)
        lsm = sps.log_softmax(t.astype(np.float64) / T, axis=-1).max(-1)
        want = np.array([lsm[n, :L].sum() for n, L in enumerate(vl)])
        np.testing.assert_allclose(r, want, rtol=1e-12, atol=1e-13)
        assert np.all(r <= 0.0) and r[2] == 0.0
        # the reference window read off the same logits as the draft is verified on: the exact form of
        # Delta (Sec. 4.3.2) reduces to the teacher-forced form, position by position
        a = oracle.score_windows(d, t, tok, mode=oracle.GREEDY, c=0.05, temperature=T, valid_len=vl)
        b = oracle.score_windows(d, t, tok, mode=oracle.GREEDY, c=0.05, temperature=T, valid_len=vl, ref_logp=r)
        np.testing.assert_allclose(a["delta"], b["delta"], rtol=1e-11, atol=1e-12)
        np.testing.assert_array_equal(a["reward_dist"], b["reward_dist"])
    # a one-hot-like row has log-probability ~0; a uniform row has -ln V
    u = np.zeros((1, 2, 64), np.float32)
    u[0, 1, 7] = 80.0
    r = oracle.reference_logprob(u)
    assert r[0] == pytest.approx(-math.log(64.0), rel=1e-12)
