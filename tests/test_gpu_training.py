"""GPU-vs-oracle parity of the training-side quantities: reverse KL and alignment divergence from the
scoring pass, group-relative advantage, sequence-form window scores with the proportional draw of a
start, expected acceptance.  Same tolerances as the scoring pass: integers bit-exact, floats within
1e-4 relative / 1e-6 absolute."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2605_14978_b200 import binding as B
from paper_2605_14978_b200 import workloads as W

from parity_util import MODES, _close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _score_with_training_outputs(x, mode, c, temperature):
    out = B.score_windows(x["draft_logits"], x["target_logits"], x["draft_tokens"], mode=MODES[mode][0], c=c,
                          temperature=temperature, uniforms=x.get("uniforms"), valid_len=x.get("valid_len"),
                          train_outputs=True)
    torch.cuda.synchronize()
    return out


def _oracle_diag(x, temperature, windows=None):
    def host(t):
        if t is None:
            return None
        return (t if windows is None else t[windows]).cpu()
    return oracle.diagnostics(host(x["draft_logits"]), host(x["target_logits"]), host(x["draft_tokens"]),
                              temperature=temperature, valid_len=host(x.get("valid_len")))


def _assert_close(name, g, o):
    g = np.asarray(g, np.float64)
    o = np.asarray(o, np.float64).astype(np.float32).astype(np.float64)   # a value beyond float32 range is +inf on both sides
    ok = _close(g, o)
    assert ok.all(), "%s: %d/%d outside tolerance, gpu=%r oracle=%r" % (name, (~ok).sum(), ok.size, g[~ok][:3], o[~ok][:3])


def _check_training_outputs(x, mode, c, temperature, windows=None):
    gpu = _score_with_training_outputs(x, mode, c, temperature)
    ref = _oracle_diag(x, temperature, windows)
    pick = (lambda t: t.cpu().numpy()) if windows is None else (lambda t: t[windows].cpu().numpy())
    for f in ("kl_rev", "kl_rev_mean", "nabla"):
        _assert_close(f, pick(gpu[f]), ref[f])
    # the normalisers against the definition: log sum exp(logit / T), float64 on the host
    tl = x["target_logits"] if windows is None else x["target_logits"][windows]
    dl = x["draft_logits"] if windows is None else x["draft_logits"][windows]
    lse_p = torch.logsumexp(tl.double() / temperature, -1).cpu().numpy()
    lse_q = torch.logsumexp(dl.double() / temperature, -1).cpu().numpy()
    vl = x.get("valid_len")
    if vl is not None:
        vl = (vl if windows is None else vl[windows]).cpu().numpy()
        keep = np.arange(lse_p.shape[1])[None, :] < vl[:, None]
        lse_p, lse_q = lse_p * keep, lse_q * keep
    _assert_close("lse_p", pick(gpu["lse_p"]), lse_p)
    _assert_close("lse_q", pick(gpu["lse_q"]), lse_q)
    # asking for the training outputs must not change the others
    base = B.score_windows(x["draft_logits"], x["target_logits"], x["draft_tokens"], mode=MODES[mode][0], c=c,
                           temperature=temperature, uniforms=x.get("uniforms"), valid_len=x.get("valid_len"))
    torch.cuda.synchronize()
    for k, v in base.items():
        if not k.startswith("_"):
            assert torch.equal(v, gpu[k]), k
    return gpu


@pytest.mark.parametrize("idx,n", [(0, 64), (1, 64), (2, 32), (3, 48), (4, 16)])
def test_reverse_kl_nabla_normalisers_on_the_workloads(idx, n):
    w = W.scaled(W.WORKLOADS[idx], n)
    x = W.generate(w, DEV)
    _check_training_outputs(x, w.modes[-1], w.c, w.temperature)


def test_reverse_kl_full_size_launch_sampled():
    w = W.WORKLOADS[2]
    x = W.generate(w, DEV)
    sample = torch.from_numpy(np.r_[0:16, 1031:1047, w.N - 16:w.N]).to(DEV)
    _check_training_outputs(x, "stochastic", w.c, w.temperature, windows=sample)


@pytest.mark.parametrize("N,K,V,dtype", [(3, 2, 8, torch.bfloat16), (5, 3, 1001, torch.bfloat16), (4, 2, 777, torch.float32),
                                         (6, 4, 32000, torch.float16), (3, 2, 1001, torch.float16),
                                         (1, 8, 128256, torch.bfloat16), (2, 32, 64, torch.bfloat16)])
def test_reverse_kl_shapes_and_paths(N, K, V, dtype):
    g = torch.Generator(device=DEV).manual_seed(N * 100 + K)
    t = torch.randn((N, K, V), generator=g, device=DEV) * 2.0
    d = t + 0.8 * torch.randn((N, K, V), generator=g, device=DEV)
    x = {"target_logits": t.to(dtype), "draft_logits": d.to(dtype),
         "draft_tokens": torch.randint(0, V, (N, K), generator=g, device=DEV, dtype=torch.int32),
         "uniforms": torch.rand((N, K), generator=g, device=DEV),
         "valid_len": torch.randint(0, K + 1, (N,), generator=g, device=DEV, dtype=torch.int32)}
    x["draft_tokens"][0, 0] = V                                   # out of range: nabla = +inf there (if valid)
    gpu = _check_training_outputs(x, "stochastic", 0.05, 0.8)
    if int(x["valid_len"][0]) > 0:
        assert float(gpu["nabla"][0, 0]) == float("inf")


def test_identical_logits_give_zero_reverse_kl_and_nabla():
    g = torch.Generator(device=DEV).manual_seed(3)
    t = (torch.randn((4, 6, 32000), generator=g, device=DEV) * 3).to(torch.bfloat16)
    x = {"target_logits": t, "draft_logits": t.clone(),
         "draft_tokens": torch.randint(0, 32000, (4, 6), generator=g, device=DEV, dtype=torch.int32),
         "uniforms": torch.rand((4, 6), generator=g, device=DEV), "valid_len": None}
    gpu = _score_with_training_outputs(x, "stochastic", 0.04, 1.0)
    assert float(gpu["kl_rev"].abs().max()) == 0.0 and float(gpu["kl_rev_mean"].abs().max()) == 0.0
    assert float(gpu["nabla"].abs().max()) == 0.0
    assert torch.equal(gpu["lse_p"], gpu["lse_q"])


# ------------------------------------------------------------------ group-relative advantage


@pytest.mark.parametrize("N,G", [(8, 8), (2048, 8), (96, 1), (100, 50), (1024, 1024), (0, 4)])
def test_group_advantage_matches_oracle(N, G):
    g = torch.Generator(device=DEV).manual_seed(N + G)
    r = torch.rand(N, generator=g, device=DEV) * 6.0
    if N >= 2 * G:
        r[:G] = 1.25                                              # a constant group
    adv = torch.full((N,), 9.0, device=DEV)
    B.ppow_group_advantage(r, G, 1e-6, adv)
    torch.cuda.synchronize()
    want = oracle.group_advantage(r.cpu().numpy().astype(np.float64), G, delta=float(np.float32(1e-6))) if N else np.zeros(0)
    _assert_close("advantage", adv.cpu().numpy(), want)
    if N >= 2 * G:
        assert float(adv[:G].abs().max()) == 0.0


def test_group_advantage_of_scored_windows_and_bad_arguments():
    w = W.scaled(W.WORKLOADS[1], 64)
    x = W.generate(w, DEV)
    out = B.score_windows(x["draft_logits"], x["target_logits"], x["draft_tokens"], mode=B.PPOW_GREEDY, c=w.c)
    adv = torch.empty_like(out["reward"])
    B.ppow_group_advantage(out["reward"], 8, 1e-4, adv)
    torch.cuda.synchronize()
    want = oracle.group_advantage(out["reward"].cpu().numpy().astype(np.float64), 8, delta=float(np.float32(1e-4)))
    _assert_close("advantage", adv.cpu().numpy(), want)
    for bad in ((out["reward"][:60], 8, 1e-4), (out["reward"], 0, 1e-4), (out["reward"], 8, -1.0), (out["reward"], 2048, 1e-4)):
        with pytest.raises(B.PpowError):
            B.ppow_group_advantage(bad[0].contiguous(), bad[1], bad[2], adv[:bad[0].numel()].contiguous())


# ------------------------------------------------------------------ sequence-form ADAW


def _sequence_case(lengths, K, seed, zero_seq=None):
    g = torch.Generator(device=DEV).manual_seed(seed)
    off = torch.tensor(np.r_[0, np.cumsum(lengths)], dtype=torch.int32, device=DEV)
    total = int(off[-1])
    v = torch.rand(total, generator=g, device=DEV) ** 4             # mostly small, a few large: like criticality scores
    if zero_seq is not None:
        v[int(off[zero_seq]):int(off[zero_seq + 1])] = 0.0
    u = torch.rand(len(lengths), generator=g, device=DEV)
    return v, off, u


@pytest.mark.parametrize("lengths,K", [([37, 10, 9, 300, 1, 2048], 10), ([5, 6, 7], 1), ([1200, 40], 33), ([64] * 50, 8)])
def test_sequence_windows_scores_and_starts_match_oracle(lengths, K):
    v, off, u = _sequence_case(lengths, K, seed=sum(lengths) + K, zero_seq=1)
    scores = torch.full_like(v, 7.0)
    starts = torch.full((len(lengths),), -5, dtype=torch.int32, device=DEV)
    B.ppow_sequence_windows(v, off, K, scores, u, starts)
    torch.cuda.synchronize()
    vh, oh, uh = v.cpu().numpy().astype(np.float64), off.cpu().numpy(), u.cpu().numpy().astype(np.float64)
    for b, T in enumerate(lengths):
        s = oracle.sliding_scores(vh[oh[b]:oh[b + 1]], K)
        got = scores[int(oh[b]):int(oh[b + 1])].cpu().numpy()
        _assert_close("scores", got[:s.size], s)
        assert np.all(got[s.size:] == 0.0)                          # no window starts in the last K-1 positions
        assert int(starts[b]) == oracle.sample_start(s, uh[b]), (b, T)   # bit-exact: same additions in the same order
    # scores only / starts only
    B.ppow_sequence_windows(v, off, K, None, u, starts)
    s2 = torch.empty_like(v)
    B.ppow_sequence_windows(v, off, K, s2, None, None)
    torch.cuda.synchronize()
    assert torch.equal(s2, scores)


def test_sequence_windows_draw_follows_the_weights():
    # one response repeated many times with different uniforms: the draws follow s_j / sum s
    K, T, reps = 4, 24, 4096
    g = torch.Generator(device=DEV).manual_seed(11)
    base = torch.rand(T, generator=g, device=DEV)
    v = base.repeat(reps)
    off = torch.arange(0, (reps + 1) * T, T, dtype=torch.int32, device=DEV)
    u = torch.rand(reps, generator=g, device=DEV)
    starts = torch.empty(reps, dtype=torch.int32, device=DEV)
    B.ppow_sequence_windows(v, off, K, None, u, starts)
    torch.cuda.synchronize()
    s = oracle.sliding_scores(base.cpu().numpy().astype(np.float64), K)
    want = np.array([oracle.sample_start(s, float(x)) for x in u.cpu().numpy().astype(np.float64)])
    np.testing.assert_array_equal(starts.cpu().numpy(), want)
    counts = np.bincount(starts.cpu().numpy(), minlength=s.size)
    assert np.abs(counts / reps - s / s.sum()).max() < 0.03


@pytest.mark.parametrize("hard_frac", [0.0, 0.2, 0.4, 0.6, 1.0])
def test_sequence_windows_mixed_draw_matches_oracle(hard_frac):
    # hard-window curriculum (App. A): ADAW draw iff the response's coin < hard_frac, uniform start otherwise
    lengths = [37, 10, 9, 300, 1, 2048, 64, 64, 64, 500, 12, 77] * 6
    K = 10
    v, off, u_draw = _sequence_case(lengths, K, seed=int(100 * hard_frac) + 5, zero_seq=1)
    g = torch.Generator(device=DEV).manual_seed(int(100 * hard_frac) + 6)
    u_mix = torch.rand(len(lengths), generator=g, device=DEV)
    if hard_frac < 1.0:                                             # coins live in [0, 1)
        u_mix[3] = float(np.float32(hard_frac))                     # the coin on the boundary: uniform branch
    scores = torch.full_like(v, 7.0)
    starts = torch.full((len(lengths),), -5, dtype=torch.int32, device=DEV)
    B.ppow_sequence_windows_mixed(v, off, K, hard_frac, scores, u_mix, u_draw, starts)
    plain_scores, plain_starts = torch.empty_like(v), torch.empty_like(starts)
    B.ppow_sequence_windows(v, off, K, plain_scores, u_draw, plain_starts)
    torch.cuda.synchronize()
    assert torch.equal(scores, plain_scores)                        # the scores do not depend on the curriculum
    vh, oh = v.cpu().numpy().astype(np.float64), off.cpu().numpy()
    um, ud = u_mix.cpu().numpy().astype(np.float64), u_draw.cpu().numpy().astype(np.float64)
    hf = float(np.float32(hard_frac))                               # the value the C ABI carries
    want = np.array([oracle.sample_start_mixed(oracle.sliding_scores(vh[oh[b]:oh[b + 1]], K), hf, um[b], ud[b])
                     for b in range(len(lengths))])
    np.testing.assert_array_equal(starts.cpu().numpy(), want)       # bit-exact
    if hard_frac == 1.0:
        assert torch.equal(starts, plain_starts)
    if 0.0 < hard_frac < 1.0:                                       # both branches were taken
        took_adaw = um < hf
        assert took_adaw.any() and (~took_adaw).any()
    for bad in (-0.1, 1.5, float("nan")):
        with pytest.raises(B.PpowError):
            B.ppow_sequence_windows_mixed(v, off, K, bad, scores, u_mix, u_draw, starts)
    with pytest.raises(B.PpowError):
        B.ppow_sequence_windows_mixed(v, off, K, 0.5, scores, None, u_draw, starts)


def test_sequence_windows_from_scored_positions():
    # criticality of a scored batch, read as one response per window row block
    w = dataclasses.replace(W.scaled(W.WORKLOADS[1], 32), V=4096)
    x = W.generate(w, DEV)
    out = B.score_windows(x["draft_logits"], x["target_logits"], x["draft_tokens"], mode=B.PPOW_GREEDY, c=w.c)
    crit = out["crit"].reshape(-1).contiguous()                     # 4 responses of 64 positions
    off = torch.arange(0, 257, 64, dtype=torch.int32, device=DEV)
    u = torch.tensor([0.0, 0.3, 0.77, 0.999], device=DEV)
    scores, starts = torch.empty_like(crit), torch.empty(4, dtype=torch.int32, device=DEV)
    B.ppow_sequence_windows(crit, off, w.K, scores, u, starts)
    torch.cuda.synchronize()
    ch = crit.cpu().numpy().astype(np.float64)
    for b in range(4):
        s = oracle.sliding_scores(ch[64 * b:64 * b + 64], w.K)
        assert int(starts[b]) == oracle.sample_start(s, float(np.float64(u[b].item())))
    with pytest.raises(B.PpowError):
        B.ppow_sequence_windows(crit, off, 0, scores, u, starts)


# ------------------------------------------------------------------ expected acceptance


@pytest.mark.parametrize("idx,n", [(0, 32), (1, 32), (3, 24)])
def test_expected_acceptance_matches_oracle(idx, n):
    w = W.scaled(W.WORKLOADS[idx], n)
    x = W.generate(w, DEV)
    gpu = _score_with_training_outputs(x, w.modes[-1], w.c, w.temperature)
    params = B.make_params(w.N, w.K, w.V, B.DTYPE_CODES[w.torch_dtype], 0, w.c, w.temperature)
    acc = torch.full((w.N, w.K), 5.0, device=DEV)
    B.ppow_expected_acceptance(params, x["draft_logits"], x["target_logits"], x["valid_len"], gpu["lse_p"], gpu["lse_q"], acc)
    torch.cuda.synchronize()
    ref = _oracle_diag(x, w.temperature)
    _assert_close("expected_accept", acc.cpu().numpy(), ref["expected_accept"])
    a = acc.cpu().numpy().astype(np.float64)
    assert np.all((a >= 0) & (a <= 1))
    kl = gpu["kl"].cpu().numpy().astype(np.float64)
    valid = np.ones_like(a, bool) if x["valid_len"] is None else (
        np.arange(w.K)[None, :] < x["valid_len"].cpu().numpy()[:, None])
    assert np.all((1.0 - a <= np.sqrt(0.5 * kl) + 1e-5)[valid])      # Pinsker (App. B.1)
    assert np.all(a[~valid] == 0.0)


def test_expected_acceptance_float16_logits():
    w = dataclasses.replace(W.scaled(W.WORKLOADS[1], 24), dtype="f16")
    x = W.generate(w, DEV)
    gpu = _score_with_training_outputs(x, "greedy", w.c, w.temperature)
    params = B.make_params(w.N, w.K, w.V, B.PPOW_F16, 0, w.c, w.temperature)
    acc = torch.empty((w.N, w.K), device=DEV)
    B.ppow_expected_acceptance(params, x["draft_logits"], x["target_logits"], None, gpu["lse_p"], gpu["lse_q"], acc)
    torch.cuda.synchronize()
    _assert_close("expected_accept", acc.cpu().numpy(), _oracle_diag(x, w.temperature)["expected_accept"])


def test_expected_acceptance_scalar_path_and_identical_distributions():
    g = torch.Generator(device=DEV).manual_seed(21)
    t = (torch.randn((3, 2, 1001), generator=g, device=DEV) * 2).to(torch.bfloat16)
    x = {"target_logits": t, "draft_logits": t.clone(),
         "draft_tokens": torch.zeros((3, 2), dtype=torch.int32, device=DEV), "uniforms": None, "valid_len": None}
    gpu = _score_with_training_outputs(x, "greedy", 0.05, 1.3)
    params = B.make_params(3, 2, 1001, B.PPOW_BF16, 0, 0.05, 1.3)
    acc = torch.empty((3, 2), device=DEV)
    B.ppow_expected_acceptance(params, x["draft_logits"], x["target_logits"], None, gpu["lse_p"], gpu["lse_q"], acc)
    torch.cuda.synchronize()
    np.testing.assert_allclose(acc.cpu().numpy(), 1.0, atol=2e-5)    # min(P, P) sums to 1


@pytest.mark.parametrize("V,off_t,off_d,dtype", [(4099, 0, 0, torch.bfloat16), (4096, 3, 3, torch.bfloat16),
                                                 (4099, 1, 1, torch.float16), (2051, 1, 1, torch.float32),
                                                 (4096, 1, 3, torch.bfloat16), (2051, 0, 2, torch.float32)])
def test_expected_acceptance_and_reference_logprob_on_rows_that_start_inside_a_unit(V, off_t, off_d, dtype):
    # odd V and base pointers off a 16-byte boundary: same offset -> vector kernels with the first and last unit of
    # a row masked; different offsets -> the scalar expected-acceptance kernel.  Huge values surround the tensors.
    N, K, T = 4, 3, 0.9
    g = torch.Generator(device=DEV).manual_seed(V + off_t + 7 * off_d)
    t = torch.randn((N, K, V), generator=g, device=DEV) * 2.0
    d = t + 0.8 * torch.randn((N, K, V), generator=g, device=DEV)
    x = {"draft_tokens": torch.randint(0, V, (N, K), generator=g, device=DEV, dtype=torch.int32), "uniforms": None,
         "valid_len": None}
    for key, val, off in (("target_logits", t, off_t), ("draft_logits", d, off_d)):
        flat = torch.full((N * K * V + 16,), 9000.0, dtype=dtype, device=DEV)
        flat[off:off + N * K * V].copy_(val.to(dtype).flatten())
        x[key] = flat[off:off + N * K * V].view(N, K, V)
    gpu = _score_with_training_outputs(x, "greedy", 0.05, T)
    params = B.make_params(N, K, V, B.DTYPE_CODES[dtype], B.PPOW_GREEDY, 0.05, T)
    acc = torch.empty((N, K), device=DEV)
    B.ppow_expected_acceptance(params, x["draft_logits"], x["target_logits"], None, gpu["lse_p"], gpu["lse_q"], acc)
    row_logp, ref_logp = torch.empty((N, K), device=DEV), torch.empty((N,), device=DEV)
    B.ppow_reference_logprob(params, x["target_logits"], None, row_logp, ref_logp)
    torch.cuda.synchronize()
    _assert_close("expected_accept", acc.cpu().numpy(), _oracle_diag(x, T)["expected_accept"])
    _assert_close("ref_logp", ref_logp.cpu().numpy(), oracle.reference_logprob(x["target_logits"].cpu(), temperature=T))


# ------------------------------------------------------------------ reference-window log-probability (exact Delta)


@pytest.mark.parametrize("N,K,V,dtype,T", [(24, 8, 32000, torch.bfloat16, 1.0), (9, 5, 1001, torch.bfloat16, 0.7),
                                           (6, 3, 5000, torch.float32, 1.3), (3, 10, 151936, torch.bfloat16, 0.7),
                                           (7, 4, 4096, torch.float16, 0.9)])
def test_reference_logprob_matches_oracle_and_feeds_the_exact_delta(N, K, V, dtype, T):
    g = torch.Generator(device=DEV).manual_seed(N + V)
    t = (torch.randn((N, K, V), generator=g, device=DEV) * 2.5).to(dtype)
    d = (t.float() + 0.6 * torch.randn((N, K, V), generator=g, device=DEV)).to(dtype)
    ref = (t.float() + 0.3 * torch.randn((N, K, V), generator=g, device=DEV)).to(dtype)   # the target on its own path
    ref[0, 0] = -3.0
    ref[0, 0, 17] = 40.0                                           # a confident row: log-probability close to 0
    tok = torch.randint(0, V, (N, K), generator=g, device=DEV, dtype=torch.int32)
    vl = torch.randint(0, K + 1, (N,), generator=g, device=DEV, dtype=torch.int32)
    vl[0] = K
    params = B.make_params(N, K, V, B.DTYPE_CODES[dtype], B.PPOW_GREEDY, 0.05, T, 1.0, 6.0)
    ref_logp = torch.full((N,), 3.0, device=DEV)
    row_logp = torch.full((N, K), 3.0, device=DEV)
    B.ppow_reference_logprob(params, ref, vl, row_logp, ref_logp)
    torch.cuda.synchronize()
    want = oracle.reference_logprob(ref.cpu(), temperature=T, valid_len=vl.cpu())
    _assert_close("ref_logp", ref_logp.cpu().numpy(), want)
    assert bool((ref_logp <= 0).all())
    rows = torch.log_softmax(ref.double() / T, -1).amax(-1) * (torch.arange(K, device=DEV)[None, :] < vl[:, None])
    _assert_close("row_logp", row_logp.cpu().numpy(), rows.cpu().numpy())
    # the exact form of Delta end to end: GPU reference log-probability into the GPU scoring pass
    gpu = B.score_windows(d, t, tok, mode=B.PPOW_GREEDY, c=0.05, temperature=T, eps=6.0, valid_len=vl, ref_logp=ref_logp)
    torch.cuda.synchronize()
    o = oracle.score_windows(d.cpu(), t.cpu(), tok.cpu(), mode=oracle.GREEDY, c=0.05, temperature=T, eps=6.0,
                             valid_len=vl.cpu(), ref_logp=want)
    _assert_close("delta", gpu["delta"].cpu().numpy(), o["delta"])
    near = np.abs(o["delta"] - 6.0) < 1e-3
    np.testing.assert_array_equal(gpu["reward_dist"].cpu().numpy()[~near], o["reward_dist"][~near].astype(np.float32))
    # reference read off the verification logits themselves: the exact form equals the teacher-forced form
    B.ppow_reference_logprob(params, t, vl, row_logp, ref_logp)
    same = B.score_windows(d, t, tok, mode=B.PPOW_GREEDY, c=0.05, temperature=T, eps=6.0, valid_len=vl, ref_logp=ref_logp)
    base = B.score_windows(d, t, tok, mode=B.PPOW_GREEDY, c=0.05, temperature=T, eps=6.0, valid_len=vl)
    torch.cuda.synchronize()
    _assert_close("delta (two forms)", same["delta"].cpu().numpy(), base["delta"].cpu().numpy().astype(np.float64))


def test_reference_logprob_bad_arguments():
    x = torch.zeros((2, 2, 64), dtype=torch.bfloat16, device=DEV)
    out, rows = torch.zeros(2, device=DEV), torch.zeros((2, 2), device=DEV)
    with pytest.raises(B.PpowError):
        B.ppow_reference_logprob(B.make_params(2, 2, 64, B.PPOW_BF16, 0, 0.05, temperature=0.0), x, None, rows, out)
    with pytest.raises(B.PpowError):
        B.ppow_reference_logprob(B.make_params(2, 0, 64, B.PPOW_BF16, 0, 0.05), x, None, rows, out)
    with pytest.raises(B.PpowError):
        B.ppow_reference_logprob(B.make_params(2, 2, 64, B.PPOW_BF16, 0, 0.05), x, None, None, out)   # row_logp is required
    B.ppow_reference_logprob(B.make_params(2, 2, 64, B.PPOW_BF16, 0, 0.05), x, None, rows, None)      # the sums are optional
    B.ppow_reference_logprob(B.make_params(0, 2, 64, B.PPOW_BF16, 0, 0.05), x, None, rows, out)       # N = 0: no-op
    torch.cuda.synchronize()
