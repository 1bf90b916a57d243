"""Helpers shared by the GPU parity tests: run both sides on the same buffers and compare.

Tolerances (stated by the build target): accepted lengths, greedy flags, argmax and selected
indices bit-exact; stochastic flags may differ only where |min(1,p/q) - u| < 1e-6; floats within
1e-4 relative / 1e-6 absolute.
"""
import numpy as np
import torch

import oracle
from paper_2605_14978_b200 import binding as B

RTOL, ATOL, BAND = 1e-4, 1e-6, 1e-6
MODES = {"greedy": (B.PPOW_GREEDY, oracle.GREEDY), "stochastic": (B.PPOW_STOCHASTIC, oracle.STOCHASTIC)}


def run_gpu(x, mode, c, temperature=1.0, eta=1.0, eps=0.5, ref_logp=None):
    out = B.score_windows(x["draft_logits"], x["target_logits"], x["draft_tokens"], mode=MODES[mode][0], c=c,
                          temperature=temperature, eta=eta, eps=eps, uniforms=x.get("uniforms"),
                          valid_len=x.get("valid_len"), ref_logp=ref_logp)
    torch.cuda.synchronize()
    return out


def run_oracle(x, mode, c, temperature=1.0, eta=1.0, eps=0.5, ref_logp=None, windows=None):
    """Oracle on host copies of the same buffers (optionally only the listed window indices)."""
    def host(t):
        if t is None:
            return None
        if windows is not None:
            t = t[windows]
        return t.detach().cpu()
    return oracle.score_windows(host(x["draft_logits"]), host(x["target_logits"]), host(x["draft_tokens"]),
                                mode=MODES[mode][1], c=c, temperature=temperature, eta=eta, eps=eps,
                                uniforms=host(x.get("uniforms")), valid_len=host(x.get("valid_len")),
                                ref_logp=None if ref_logp is None else host(ref_logp).double())


def _close(g, o):
    g = np.asarray(g, np.float64)
    o = np.asarray(o, np.float64)
    both_inf = np.isinf(g) & np.isinf(o) & (np.sign(g) == np.sign(o))
    with np.errstate(invalid="ignore"):
        ok = np.abs(g - o) <= ATOL + RTOL * np.abs(o)
    return ok | both_inf


def compare_scores(gpu, ref, mode, uniforms, eps=0.5, windows=None):
    """Element-by-element comparison.  Returns a dict of counts; raises AssertionError on a mismatch."""
    def g(name):
        t = gpu[name]
        if windows is not None:
            t = t[windows]
        return t.detach().cpu().numpy()

    np.testing.assert_array_equal(g("target_argmax"), ref["target_argmax"], err_msg="target_argmax")
    for f in ("kl", "conf", "crit", "logp_tok", "logq_tok"):
        ok = _close(g(f), ref[f])
        assert ok.all(), "%s: %d/%d outside tolerance, worst gpu=%r oracle=%r" % (
            f, (~ok).sum(), ok.size, g(f)[~ok][:3], ref[f][~ok][:3])

    flags_g, flags_o = g("accept_flag"), ref["accept_flag"]
    differ = flags_g != flags_o
    band_windows = np.zeros(flags_g.shape[0], bool)
    if mode == "greedy":
        assert not differ.any(), "greedy accept flags differ at %d positions" % differ.sum()
    else:
        u = uniforms if windows is None else uniforms[windows]
        u = u.detach().cpu().numpy().astype(np.float64)
        in_band = np.abs(ref["alpha"] - u) < BAND
        assert not (differ & ~in_band).any(), "stochastic flags differ outside the 1e-6 band at %d positions" % (
            (differ & ~in_band).sum())
        band_windows = differ.any(axis=1)
    keep = ~band_windows
    np.testing.assert_array_equal(g("accepted_len")[keep], ref["accepted_len"][keep], err_msg="accepted_len")
    for f in ("reward_speedup", "delta", "score"):
        ok = _close(g(f)[keep], ref[f][keep])
        assert ok.all(), "%s: %d outside tolerance" % (f, (~ok).sum())
    # reward_dist is a threshold on delta: windows whose delta sits on the threshold are not compared
    near_eps = np.abs(ref["delta"] - eps) <= ATOL + RTOL * abs(eps)
    k2 = keep & ~near_eps
    np.testing.assert_array_equal(g("reward_dist")[k2], ref["reward_dist"][k2].astype(np.float32), err_msg="reward_dist")
    assert _close(g("reward")[k2], ref["reward"][k2]).all(), "reward"
    return {"band_flag_differences": int(differ.sum()), "windows_skipped": int(band_windows.sum() + (near_eps & keep).sum())}


def compare_selection(gpu_scores, n_keep, oracle_scores=None):
    """(i) GPU selection against the oracle's selection on the identical float32 scores: bit-exact.
    (ii) if oracle float64 scores are given: the two selections may differ only in windows whose
    oracle score is within tolerance of the cut."""
    sel, mask = B.select_windows(gpu_scores, n_keep, want_mask=True)
    torch.cuda.synchronize()
    sel = sel.cpu().numpy()
    mask = mask.cpu().numpy()
    s32 = gpu_scores.detach().cpu().numpy()
    want, want_mask = oracle.select_windows(s32.astype(np.float64), n_keep, want_mask=True)
    np.testing.assert_array_equal(sel, want, err_msg="selected indices on identical scores")
    np.testing.assert_array_equal(mask, want_mask, err_msg="selection mask")
    swapped = 0
    if oracle_scores is not None and 0 < n_keep < len(oracle_scores):
        ref_sel = oracle.select_windows(oracle_scores, n_keep)
        cut = oracle_scores[ref_sel[-1]]
        sym = set(sel.tolist()) ^ set(ref_sel.tolist())
        for i in sym:
            assert abs(oracle_scores[i] - cut) <= 2 * (ATOL + RTOL * abs(cut)), (
                "window %d selected by one side only and not near the cut" % i)
        swapped = len(sym)
    return {"near_cut_swaps": swapped}
