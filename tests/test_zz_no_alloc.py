"""ppow_score_windows_noalloc: the scoring entry point for callers that cannot allocate scratch.

Some users of the library sit beside a framework that has already claimed the device's memory and
whose allocator they cannot reach (a plain-C plugin, a scheduler thread), or must not allocate once
a run has started.  They call this entry point, which uses a fixed 4 MiB array inside the library
instead of a caller-provided workspace.  The test calls it through the C ABI twice in a row (the
array is shared and keeps the previous call's contents) and compares every output with the ordinary
entry point and with the float64 oracle; the headline shape, the largest that fits the array, goes
through it once; and the call's error word is read back.  Collected last on purpose.
"""
import dataclasses
import os
import sys

import numpy as np
import pytest
import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

from paper_2605_14978_b200 import binding as B
from paper_2605_14978_b200 import workloads as W
from parity_util import compare_scores, run_oracle

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _reference(params, x):
    out = B.alloc_outputs(params.N, params.K, DEV)
    ws = B.alloc_workspace(B.ppow_score_workspace_bytes(params), DEV)
    B.ppow_score_windows(params, x["draft_logits"], x["target_logits"], x["draft_tokens"], x["uniforms"],
                         x["valid_len"], None, out, ws)
    torch.cuda.synchronize()
    return out


def test_noalloc_entry_point_matches_workspace_entry_point_twice_in_a_row():
    # two different problems back to back: the second call finds the first call's leftovers in the array
    w1 = dataclasses.replace(W.scaled(W.WORKLOADS[3], 96), V=8 * 1251)       # ragged lengths, stochastic
    w2 = dataclasses.replace(W.scaled(W.WORKLOADS[1], 40), V=32000)          # greedy, more rows per window
    cases = []
    for w, mode in ((w1, B.PPOW_STOCHASTIC), (w2, B.PPOW_GREEDY)):
        x = W.generate(w, DEV)
        params = B.make_params(w.N, w.K, w.V, B.PPOW_BF16, mode, w.c, w.temperature)
        assert 0 < B.ppow_score_workspace_bytes(params) <= B.ppow_noalloc_scratch_bytes()
        name = "stochastic" if mode == B.PPOW_STOCHASTIC else "greedy"
        cases.append((params, x, _reference(params, x), name, run_oracle(x, name, w.c, w.temperature)))
    for _ in range(2):                                                        # and the whole sequence again
        for params, x, want, name, ref in cases:
            got = {k: torch.full_like(v, 77) for k, v in want.items()}       # poisoned, preallocated outputs
            B.ppow_score_windows_noalloc(params, x["draft_logits"], x["target_logits"], x["draft_tokens"],
                                         x["uniforms"], x["valid_len"], None, got)
            torch.cuda.synchronize()
            for k in want:
                if want[k].dtype.is_floating_point:
                    torch.testing.assert_close(got[k], want[k], rtol=1e-4, atol=1e-6, equal_nan=True, msg=k)
                else:
                    assert torch.equal(got[k], want[k]), k
            compare_scores(got, ref, name, x["uniforms"])                     # and against the oracle itself
            assert B.ppow_noalloc_read_error_flags() == (B.PPOW_OK, 0)


def test_noalloc_entry_point_on_the_headline_shape_against_the_oracle():
    # 2048 x 8 x 128256: the workload the built-in array was sized for
    w = W.WORKLOADS[2]
    x = W.generate(w, DEV)
    params = B.make_params(w.N, w.K, w.V, B.PPOW_BF16, B.PPOW_STOCHASTIC, w.c, w.temperature)
    assert B.ppow_score_workspace_bytes(params) <= B.ppow_noalloc_scratch_bytes()
    got = B.alloc_outputs(w.N, w.K, DEV)
    B.ppow_score_windows_noalloc(params, x["draft_logits"], x["target_logits"], x["draft_tokens"], x["uniforms"],
                                 x["valid_len"], None, got)
    torch.cuda.synchronize()
    sample = torch.from_numpy(np.r_[0:16, 1031:1047, w.N - 16:w.N]).to(DEV)
    ref = run_oracle(x, "stochastic", w.c, w.temperature, windows=sample)
    compare_scores(got, ref, "stochastic", x["uniforms"], windows=sample)
    assert B.ppow_noalloc_read_error_flags() == (B.PPOW_OK, 0)


def test_noalloc_entry_point_reports_an_out_of_range_token_through_its_own_error_word():
    w = dataclasses.replace(W.scaled(W.WORKLOADS[1], 8), V=4096)
    x = W.generate(w, DEV)
    x["draft_tokens"][3, 2] = w.V + 5
    params = B.make_params(w.N, w.K, w.V, B.PPOW_BF16, B.PPOW_GREEDY, w.c)
    got = B.alloc_outputs(w.N, w.K, DEV)
    B.ppow_score_windows_noalloc(params, x["draft_logits"], x["target_logits"], x["draft_tokens"], None, None, None, got)
    status, flags = B.ppow_noalloc_read_error_flags()
    assert status == B.PPOW_OK and flags == B.PPOW_FLAG_TOKEN_RANGE
    assert int(got["accept_flag"][3, 2]) == 0 and torch.isinf(got["logp_tok"][3, 2])
    x["draft_tokens"][3, 2] = 0                                               # the next call clears the word
    B.ppow_score_windows_noalloc(params, x["draft_logits"], x["target_logits"], x["draft_tokens"], None, None, None, got)
    assert B.ppow_noalloc_read_error_flags() == (B.PPOW_OK, 0)


def test_noalloc_entry_point_refuses_requests_beyond_its_scratch():
    big = B.make_params(8192, 12, 152064, B.PPOW_BF16, B.PPOW_GREEDY, 0.03)
    assert B.ppow_score_workspace_bytes(big) > B.ppow_noalloc_scratch_bytes()
    dummy = torch.zeros(8, dtype=torch.bfloat16, device=DEV)
    tok = torch.zeros(8, dtype=torch.int32, device=DEV)
    out = {"accepted_len": torch.zeros(8, dtype=torch.int32, device=DEV)}
    with pytest.raises(B.PpowError) as e:                                     # refused before anything is launched
        B.ppow_score_windows_noalloc(big, dummy, dummy, tok, None, None, None, out)
    assert e.value.status == B.PPOW_ERR_UNSUPPORTED
    for bad in (B.make_params(4, 4, 1, B.PPOW_BF16, B.PPOW_GREEDY, 0.03),
                B.make_params(0, 4, 1, B.PPOW_BF16, B.PPOW_GREEDY, 0.03)):    # invalid V, also when there is nothing to score
        with pytest.raises(B.PpowError) as e:
            B.ppow_score_windows_noalloc(bad, dummy, dummy, tok, None, None, None, out)
        assert e.value.status == B.PPOW_ERR_INVALID_ARG
