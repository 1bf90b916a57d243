"""Pins of the float64 oracle against things other than itself: library routines, closed forms,
values and worked examples printed in the paper, brute force and invariants (CPU only)."""
import math
import os

import numpy as np
import pytest
import scipy.special as sps
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_case(rng, N, K, V, sigma=0.7, dtype=np.float32):
    t = (rng.normal(size=(N, K, V)) * 2.0).astype(dtype)
    d = (t + sigma * rng.normal(size=(N, K, V))).astype(dtype)
    tok = rng.integers(0, V, size=(N, K)).astype(np.int32)
    u = rng.random((N, K), dtype=np.float32)
    return d, t, tok, u


def _to_bf16_bits(x):
    return torch.from_numpy(x).to(torch.bfloat16)


# ---------------------------------------------------------------- softmax / entropy / KL


@pytest.mark.parametrize("T", [1.0, 0.7, 2.5])
@pytest.mark.parametrize("V", [2, 17, 1000])
def test_entropy_kl_logprobs_match_scipy(T, V):
    rng = np.random.default_rng(V * 7 + int(T * 10))
    d, t, tok, u = _rand_case(rng, 5, 3, V)
    o = oracle.score_windows(d, t, tok, mode=oracle.STOCHASTIC, c=0.05, temperature=T, uniforms=u)
    P = sps.softmax(t.astype(np.float64) / T, axis=-1)
    Q = sps.softmax(d.astype(np.float64) / T, axis=-1)
    lse_t = sps.logsumexp(t.astype(np.float64) / T, axis=-1)
    lse_d = sps.logsumexp(d.astype(np.float64) / T, axis=-1)
    H = sps.entr(P).sum(-1)
    KL = sps.rel_entr(P, Q).sum(-1)
    np.testing.assert_allclose(o["entropy"], H, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(o["kl"], KL, rtol=1e-9, atol=1e-13)
    np.testing.assert_allclose(o["conf"], 1.0 - H / math.log(V), rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(o["crit"], (1.0 - H / math.log(V)) * KL, rtol=1e-9, atol=1e-13)
    lp = np.take_along_axis(t.astype(np.float64) / T, tok[..., None].astype(np.int64), -1)[..., 0] - lse_t
    lq = np.take_along_axis(d.astype(np.float64) / T, tok[..., None].astype(np.int64), -1)[..., 0] - lse_d
    np.testing.assert_allclose(o["logp_tok"], lp, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(o["logq_tok"], lq, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(o["alpha"], np.minimum(1.0, np.exp(lp - lq)), rtol=1e-11)
    np.testing.assert_array_equal(o["target_argmax"], t.argmax(-1))
    np.testing.assert_allclose(o["logp_max"], (t.astype(np.float64) / T).max(-1) - lse_t, rtol=1e-12, atol=1e-12)


def test_kl_matches_torch_float64_on_bf16_storage():
    rng = np.random.default_rng(3)
    d, t, tok, u = _rand_case(rng, 4, 2, 333)
    db, tb = _to_bf16_bits(d), _to_bf16_bits(t)
    o = oracle.score_windows(db, tb, tok, mode=oracle.GREEDY, c=0.05)
    lp = torch.log_softmax(tb.to(torch.float64), -1)
    lq = torch.log_softmax(db.to(torch.float64), -1)
    kl = torch.nn.functional.kl_div(lq, lp, log_target=True, reduction="none").sum(-1)
    np.testing.assert_allclose(o["kl"], kl.numpy(), rtol=1e-9, atol=1e-13)
    ent = -(lp.exp() * lp).sum(-1)
    np.testing.assert_allclose(o["entropy"], ent.numpy(), rtol=1e-11)
    # argmax on the stored bf16 values, lowest index on ties (bf16 ties are common)
    tf = tb.to(torch.float64).numpy()
    expect = np.array([[int(np.flatnonzero(r == r.max())[0]) for r in w] for w in tf])
    np.testing.assert_array_equal(o["target_argmax"], expect)


def test_two_symbol_closed_form_fixes_direction_and_operands():
    # target logits (0, ln 3) => P = (1/4, 3/4); draft logits (0, 0) => Q = (1/2, 1/2)
    t = np.array([[[0.0, math.log(3.0)]]], np.float32)
    d = np.array([[[0.0, 0.0]]], np.float32)
    tok = np.array([[1]], np.int32)
    o = oracle.score_windows(d, t, tok, mode=oracle.STOCHASTIC, c=0.1, uniforms=np.array([[0.9]], np.float32))
    p1 = math.exp(float(np.float32(math.log(3.0))))
    P = np.array([1.0, p1]) / (1.0 + p1)
    H = -(P * np.log(P)).sum()
    KL_pq = (P * np.log(P / 0.5)).sum()
    KL_qp = (0.5 * np.log(0.5 / P)).sum()
    assert abs(KL_pq - (0.25 * math.log(0.5) + 0.75 * math.log(1.5))) < 1e-7
    assert abs(KL_pq - KL_qp) > 1e-2                       # the two directions differ on this case
    assert o["kl"][0, 0] == pytest.approx(KL_pq, rel=1e-12)
    assert o["entropy"][0, 0] == pytest.approx(H, rel=1e-12)
    assert o["conf"][0, 0] == pytest.approx(1.0 - H / math.log(2.0), rel=1e-12)
    assert o["logp_tok"][0, 0] == pytest.approx(math.log(P[1]), rel=1e-12)
    assert o["logq_tok"][0, 0] == pytest.approx(math.log(0.5), rel=1e-12)
    assert o["alpha"][0, 0] == 1.0 and o["accept_flag"][0, 0] == 1   # p/q = 1.5 -> min(1, .) = 1
    # the other token: p/q = 0.5; accept iff u <= 0.5
    for u, want in ((0.49, 1), (0.51, 0)):
        o2 = oracle.score_windows(d, t, np.array([[0]], np.int32), mode=oracle.STOCHASTIC, c=0.1,
                                  uniforms=np.array([[u]], np.float32))
        assert o2["alpha"][0, 0] == pytest.approx(P[0] / 0.5, rel=1e-12)
        assert o2["accept_flag"][0, 0] == want
    # the test is u <= alpha, not u < alpha: P = (1/2, 1/2), Q = (1, 0) to double precision => alpha = 1/2
    t2 = np.zeros((1, 1, 2), np.float32)
    d2 = np.array([[[0.0, -200.0]]], np.float32)
    for u, want in ((0.5, 1), (np.nextafter(np.float32(0.5), np.float32(1.0)), 0)):
        o3 = oracle.score_windows(d2, t2, np.array([[0]], np.int32), mode=oracle.STOCHASTIC, c=0.1,
                                  uniforms=np.array([[u]], np.float32))
        assert o3["alpha"][0, 0] == 0.5
        assert o3["accept_flag"][0, 0] == want


def test_uniform_target_has_zero_confidence():
    V = 50
    t = np.zeros((1, 2, V), np.float32)
    d = np.random.default_rng(0).normal(size=(1, 2, V)).astype(np.float32)
    o = oracle.score_windows(d, t, np.zeros((1, 2), np.int32), mode=oracle.GREEDY, c=0.05)
    np.testing.assert_allclose(o["entropy"], math.log(V), rtol=1e-13)
    np.testing.assert_allclose(o["conf"], 0.0, atol=1e-13)
    np.testing.assert_allclose(o["crit"], 0.0, atol=1e-12)
    assert np.all(o["kl"] > 0)


def test_one_hot_target_has_full_confidence():
    V = 64
    t = np.full((1, 1, V), -200.0, np.float32)
    t[0, 0, 5] = 0.0
    d = np.zeros((1, 1, V), np.float32)
    o = oracle.score_windows(d, t, np.array([[5]], np.int32), mode=oracle.GREEDY, c=0.05)
    assert o["entropy"][0, 0] < 1e-80
    assert o["conf"][0, 0] == pytest.approx(1.0)
    assert o["kl"][0, 0] == pytest.approx(math.log(V), rel=1e-12)   # KL(one-hot || uniform) = ln V


def test_identical_distributions_zero_divergence_full_stochastic_acceptance():
    rng = np.random.default_rng(11)
    d, t, tok, u = _rand_case(rng, 6, 5, 97)
    o = oracle.score_windows(t, t, tok, mode=oracle.STOCHASTIC, c=0.05, uniforms=u)
    assert np.all(o["kl"] == 0.0)
    assert np.all(o["crit"] == 0.0) and np.all(o["score"] == 0.0)
    assert np.all(o["alpha"] == 1.0)
    assert np.all(o["accept_flag"] == 1)
    assert np.all(o["accepted_len"] == 5)
    # greedy: full acceptance needs the drafted token to be the mode
    o = oracle.score_windows(t, t, t.argmax(-1).astype(np.int32), mode=oracle.GREEDY, c=0.05)
    assert np.all(o["accepted_len"] == 5)
    assert np.all(o["delta"] == 0.0)


def test_invariants_ranges_pinsker_and_shift():
    rng = np.random.default_rng(5)
    d, t, tok, u = _rand_case(rng, 8, 4, 200, sigma=1.5)
    o = oracle.score_windows(d, t, tok, mode=oracle.STOCHASTIC, c=0.05, uniforms=u)
    assert np.all(o["kl"] >= 0) and np.all(o["conf"] >= 0) and np.all(o["conf"] <= 1)
    assert np.all(o["alpha"] > 0) and np.all(o["alpha"] <= 1)
    P = sps.softmax(t.astype(np.float64), -1)
    Q = sps.softmax(d.astype(np.float64), -1)
    tv = 0.5 * np.abs(P - Q).sum(-1)
    assert np.all(tv <= np.sqrt(o["kl"] / 2.0) + 1e-12)          # Pinsker (App. B.1)
    assert np.all((o["accepted_len"] >= 0) & (o["accepted_len"] <= 4))
    # adding a constant to a row changes nothing (use an exactly representable shift)
    o2 = oracle.score_windows(d + np.float32(8.0), t - np.float32(16.0), tok, mode=oracle.STOCHASTIC, c=0.05,
                              uniforms=u)
    for f in ("kl", "entropy", "crit", "logp_tok", "logq_tok", "alpha", "score", "delta"):
        np.testing.assert_allclose(o2[f], o[f], rtol=1e-5, atol=1e-6)   # inputs re-rounded to f32 by the shift
    # logits*T at temperature T are the logits at temperature 1 (T a power of two: exact)
    o3 = oracle.score_windows(d * np.float32(4.0), t * np.float32(4.0), tok, mode=oracle.STOCHASTIC, c=0.05,
                              temperature=4.0, uniforms=u)
    for f in oracle.ppow_oracle.POSITION_FIELDS + oracle.ppow_oracle.WINDOW_FIELDS:
        np.testing.assert_array_equal(o3[f], o[f])


def test_monte_carlo_acceptance_rate_is_one_minus_tv():
    # App. B.1: with yhat ~ Q and u ~ U(0,1), P[accept] = sum_v min(P, Q) = 1 - TV(P, Q)
    rng = np.random.default_rng(2)
    V, M = 12, 40000
    t1 = (rng.normal(size=V) * 1.5).astype(np.float32)
    d1 = (t1 + rng.normal(size=V)).astype(np.float32)
    P = sps.softmax(t1.astype(np.float64))
    Q = sps.softmax(d1.astype(np.float64))
    expect = np.minimum(P, Q).sum()
    tok = rng.choice(V, size=(M, 1), p=Q).astype(np.int32)
    u = rng.random((M, 1), dtype=np.float32)
    t = np.broadcast_to(t1, (M, 1, V)).copy()
    d = np.broadcast_to(d1, (M, 1, V)).copy()
    o = oracle.score_windows(d, t, tok, mode=oracle.STOCHASTIC, c=0.05, uniforms=u)
    rate = o["accept_flag"].mean()
    sigma = math.sqrt(expect * (1 - expect) / M)
    assert abs(rate - expect) < 4.5 * sigma
    assert abs(o["accepted_len"].mean() - expect) < 4.5 * sigma   # K = 1: tau is the flag


# ---------------------------------------------------------------- acceptance, prefix, rewards


def _one_hot_logits(ids, V, hi=10.0):
    x = np.zeros((1, len(ids), V), np.float32)
    for t, i in enumerate(ids):
        x[0, t, i] = hi
    return x


def _read_fig1():
    rows = {}
    with open(os.path.join(GOLDEN, "fig1_examples.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            head, target, k = line.split("|")
            head = head.split()
            rows[head[0]] = (int(head[1]), [int(x) for x in head[2:]], [int(x) for x in target.split()], int(k))
    return rows


def test_fig1_worked_examples():
    ex = _read_fig1()
    V, gamma = 16, 0.12
    K, draft, target, k = ex["a"]
    t = _one_hot_logits(target, V)
    o = oracle.score_windows(t.copy(), t, np.array([draft], np.int32), mode=oracle.GREEDY, c=gamma)
    assert o["accepted_len"][0] == k == 3
    np.testing.assert_array_equal(o["accept_flag"][0], [1, 1, 1, 0, 0])
    assert o["reward_speedup"][0] == pytest.approx(3 / (3 * gamma + 1))
    assert o["reward_dist"][0] == 0.0                 # active only when k = 0

    K, draft, target, k = ex["b"]
    # target nearly indifferent between its own token and the drafted one: small Delta
    t = _one_hot_logits(target, V, hi=6.0)
    for pos, tokd in enumerate(draft):
        t[0, pos, tokd] = 6.0 - 0.05
    o = oracle.score_windows(t.copy(), t, np.array([draft], np.int32), mode=oracle.GREEDY, c=gamma, eta=1.0,
                             eps=0.5)
    assert o["accepted_len"][0] == k == 0
    assert o["reward_speedup"][0] == 0.0
    assert o["delta"][0] == pytest.approx(5 * 0.05, rel=1e-5)
    assert o["reward_dist"][0] == 1.0 and o["reward"][0] == 1.0
    # a drafted window the target finds much less likely: no credit
    t2 = _one_hot_logits(target, V, hi=6.0)
    o = oracle.score_windows(t2.copy(), t2, np.array([draft], np.int32), mode=oracle.GREEDY, c=gamma)
    assert o["accepted_len"][0] == 0 and o["delta"][0] == pytest.approx(30.0) and o["reward"][0] == 0.0


def test_reward_speedup_matches_printed_column():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "reward_speedup_table.txt")) if l[0] != "#"]
    ks = [int(r[0]) for r in rows]
    printed = [float(r[1]) for r in rows]
    gamma, V, K = 0.1247, 4, 7
    # window k accepts exactly its first k tokens (token 0 is the target mode everywhere)
    t = np.zeros((K + 1, K, V), np.float32)
    t[:, :, 0] = 5.0
    tok = np.ones((K + 1, K), np.int32)
    for k in range(K + 1):
        tok[k, :k] = 0
    o = oracle.score_windows(t.copy(), t, tok, mode=oracle.GREEDY, c=gamma)
    np.testing.assert_array_equal(o["accepted_len"], np.arange(K + 1))
    assert o["reward_speedup"][0] == 0.0
    for k, p in zip(ks, printed):
        assert round(o["reward_speedup"][k], 2) == pytest.approx(p, abs=1e-9)
    r = o["reward_speedup"]
    assert np.all(np.diff(r) > 0) and np.all(r < 1.0 / gamma)      # strictly increasing, bounded by 1/gamma
    # the rounded gamma of the hyperparameter table does not reproduce the column
    assert round(2 / (2 * 0.12 + 1), 2) != 1.60


@pytest.mark.parametrize("K", [1, 5, 12])
def test_accepted_length_brute_force_all_patterns(K):
    N, V = 2 ** K, 4
    pat = ((np.arange(N)[:, None] >> np.arange(K)[None, :]) & 1).astype(np.uint8)   # every flag pattern
    t = np.zeros((N, K, V), np.float32)
    t[:, :, 2] = 3.0                                        # target mode is token 2
    tok = np.where(pat == 1, 2, 1).astype(np.int32)
    rng = np.random.default_rng(K)
    L = rng.integers(0, K + 1, size=N).astype(np.int32)
    for valid in (None, L):
        o = oracle.score_windows(t.copy(), t, tok, mode=oracle.GREEDY, c=0.05, valid_len=valid)
        for n in range(N):
            Ln = K if valid is None else int(L[n])
            np.testing.assert_array_equal(o["accept_flag"][n, :Ln], pat[n, :Ln])
            assert np.all(o["accept_flag"][n, Ln:] == 0)
            first_zero = next((i for i in range(Ln) if pat[n, i] == 0), Ln)
            assert o["accepted_len"][n] == first_zero == oracle.tau_cumprod(pat[n, :Ln])
            assert 0 <= o["accepted_len"][n] <= Ln


def test_rewards_delta_and_score_definitions():
    rng = np.random.default_rng(9)
    N, K, V = 40, 6, 30
    d, t, tok, u = _rand_case(rng, N, K, V, sigma=0.4)
    tok[:10] = t[:10].argmax(-1)                            # some windows draft the target mode everywhere
    L = rng.integers(0, K + 1, size=N).astype(np.int32)
    c, eta, eps = 0.07, 0.8, 10.0
    o = oracle.score_windows(d, t, tok, mode=oracle.STOCHASTIC, c=c, eta=eta, eps=eps, uniforms=u, valid_len=L)
    for n in range(N):
        Ln = int(L[n])
        if Ln == 0:
            for f in oracle.ppow_oracle.WINDOW_FIELDS:
                assert o[f][n] == 0
            continue
        k = int(o["accepted_len"][n])
        assert o["reward_speedup"][n] == pytest.approx(k / (k * c + 1), rel=1e-14)
        gap = (o["logp_max"][n, :Ln] - o["logp_tok"][n, :Ln])
        assert np.all(gap >= 0)
        assert o["delta"][n] == pytest.approx(gap.sum(), rel=1e-12, abs=1e-14)
        assert (o["delta"][n] == 0) == bool(np.all(tok[n, :Ln] == o["target_argmax"][n, :Ln]))
        want_dist = eta if (k == 0 and o["delta"][n] < eps) else 0.0
        assert o["reward_dist"][n] == want_dist
        assert o["reward"][n] == pytest.approx(o["reward_speedup"][n] + want_dist)   # Alg. 1: total reward
        assert o["score"][n] == pytest.approx(o["crit"][n, :Ln].mean(), rel=1e-12)   # s = mean of v_t
        assert np.all(o["crit"][n, Ln:] == 0) and np.all(o["accept_flag"][n, Ln:] == 0)
    assert (o["reward_dist"] > 0).any() and (o["reward_dist"] == 0).any()
    # caller-supplied log-probability of the target's own reference window
    ref = rng.normal(size=N) - 3.0
    o2 = oracle.score_windows(d, t, tok, mode=oracle.STOCHASTIC, c=c, eta=eta, eps=eps, uniforms=u, valid_len=L,
                              ref_logp=ref)
    for n in range(N):
        if L[n] > 0:
            assert o2["delta"][n] == pytest.approx(ref[n] - o["logp_tok"][n, :L[n]].sum(), rel=1e-12)


def test_out_of_vocabulary_tokens_are_rejected():
    rng = np.random.default_rng(1)
    d, t, tok, u = _rand_case(rng, 2, 3, 9)
    tok[0, 1] = 9
    tok[1, 0] = -1
    for mode in (oracle.GREEDY, oracle.STOCHASTIC):
        o = oracle.score_windows(d, t, tok, mode=mode, c=0.05, uniforms=np.zeros((2, 3), np.float32))
        assert o["accept_flag"][0, 1] == 0 and o["accept_flag"][1, 0] == 0
        assert o["accepted_len"][0] <= 1 and o["accepted_len"][1] == 0
        assert o["logp_tok"][0, 1] == -np.inf and o["alpha"][0, 1] == 0.0
        assert o["delta"][0] == np.inf and o["reward_dist"][1] == 0.0


def test_heavy_tailed_rows_stay_finite():
    rng = np.random.default_rng(4)
    t = (rng.standard_t(3, size=(3, 2, 500)) * 300).astype(np.float32)
    d = (t + rng.standard_t(3, size=t.shape) * 100).astype(np.float32)
    tok = rng.integers(0, 500, size=(3, 2)).astype(np.int32)
    o = oracle.score_windows(d, t, tok, mode=oracle.STOCHASTIC, c=0.03, uniforms=rng.random((3, 2), dtype=np.float32))
    for f in ("kl", "entropy", "conf", "crit", "alpha", "score", "logp_tok", "logq_tok"):
        assert np.all(np.isfinite(o[f])), f
    assert np.all(o["kl"] >= -1e-15) and np.all(o["conf"] <= 1.0)   # rounding may leave -1e-100


# ---------------------------------------------------------------- selection


def test_selection_matches_python_sorted_and_tie_rules():
    rng = np.random.default_rng(6)
    for N, n_keep in ((1, 1), (10, 3), (257, 64), (1000, 1000), (50, 0)):
        s = rng.random(N)
        s[rng.integers(0, N, size=N // 3)] = 0.5            # plant exact ties
        sel, mask = oracle.select_windows(s, n_keep, want_mask=True)
        want = sorted(range(N), key=lambda i: (-s[i], i))[:n_keep]
        np.testing.assert_array_equal(sel, want)
        assert mask.sum() == n_keep and np.all(mask[want] == 1)
    np.testing.assert_array_equal(oracle.select_windows(np.full(20, 3.0), 7), np.arange(7))
    # shuffling windows with distinct scores permutes the selected set
    s = rng.permutation(100).astype(np.float64)
    perm = rng.permutation(100)
    a = set(oracle.select_windows(s, 25).tolist())
    b = set(perm[oracle.select_windows(s[perm], 25)].tolist())
    assert a == b == set(np.argsort(-s)[:25].tolist())
    with pytest.raises(RuntimeError):
        oracle.select_windows(s, 101)


def test_oracle_rejects_bad_arguments():
    d = np.zeros((1, 1, 4), np.float32)
    tok = np.zeros((1, 1), np.int32)
    with pytest.raises(RuntimeError):
        oracle.score_windows(d, d, tok, mode=oracle.STOCHASTIC, c=0.05)             # no uniforms
    with pytest.raises(RuntimeError):
        oracle.score_windows(d, d, tok, mode=oracle.GREEDY, c=0.05, temperature=0.0)
    with pytest.raises(RuntimeError):
        oracle.score_windows(d[:, :, :1], d[:, :, :1], tok, mode=oracle.GREEDY, c=0.05)   # V = 1: log|V| = 0


def test_thread_count_does_not_change_results():
    rng = np.random.default_rng(8)
    d, t, tok, u = _rand_case(rng, 13, 3, 50)
    a = oracle.score_windows(d, t, tok, mode=oracle.STOCHASTIC, c=0.05, uniforms=u, n_threads=1)
    b = oracle.score_windows(d, t, tok, mode=oracle.STOCHASTIC, c=0.05, uniforms=u, n_threads=5)
    for f in a:
        np.testing.assert_array_equal(a[f], b[f])


def test_storage_decoders_are_exact_on_every_bit_pattern():
    bits = np.arange(65536, dtype=np.uint16)
    half = bits.view(np.float16)
    finite = np.isfinite(half)
    got = oracle.decode(half)
    np.testing.assert_array_equal(got[finite], half[finite].astype(np.float64))          # all 63488 finite halves
    assert np.all(np.isinf(got[np.isinf(half)])) and np.all(np.isnan(got[np.isnan(half)]))
    assert np.array_equal(np.signbit(got[finite]), np.signbit(half[finite]))             # -0.0 keeps its sign
    bf = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
    want = bf.to(torch.float64).numpy()
    ok = np.isfinite(want)
    np.testing.assert_array_equal(oracle.decode(bits)[ok], want[ok])                      # all finite bf16 patterns
    f = np.array([0.0, -0.0, 1.0, -3.5, 1e-38, 3.4e38, 1.17549435e-38 / 4], np.float32)
    np.testing.assert_array_equal(oracle.decode(f), f.astype(np.float64))


def test_float16_logits_score_like_their_float32_values():
    rng = np.random.default_rng(41)
    d, t, tok, u = _rand_case(rng, 4, 3, 200)
    dh, th = d.astype(np.float16), t.astype(np.float16)
    a = oracle.score_windows(dh, th, tok, mode=oracle.STOCHASTIC, c=0.05, temperature=0.8, uniforms=u)
    b = oracle.score_windows(dh.astype(np.float32), th.astype(np.float32), tok, mode=oracle.STOCHASTIC, c=0.05,
                             temperature=0.8, uniforms=u)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])
