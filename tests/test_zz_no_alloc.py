"""ppow_score_windows_noalloc: the scoring entry point for callers that cannot allocate scratch.

Some users of the library sit beside a framework that has already claimed the device's memory and
whose allocator they cannot reach (a plain-C plugin, a scheduler thread), or must not allocate once
a run has started.  They call this entry point, which uses a fixed 4 MiB array inside the library
instead of a caller-provided workspace.  The test calls it through the C ABI twice in a row (the
array is shared and keeps the previous call's contents) and compares every output with the ordinary
entry point, which is itself checked against the oracle elsewhere.  Collected last on purpose.
"""
import dataclasses

import pytest
import torch

from paper_2605_14978_b200 import binding as B
from paper_2605_14978_b200 import workloads as W

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
        cases.append((params, x, _reference(params, x)))
    for _ in range(2):                                                        # and the whole sequence again
        for params, x, want in cases:
            got = {k: torch.full_like(v, 77) for k, v in want.items()}       # poisoned, preallocated outputs
            B.ppow_score_windows_noalloc(params, x["draft_logits"], x["target_logits"], x["draft_tokens"],
                                         x["uniforms"], x["valid_len"], None, got)
            torch.cuda.synchronize()
            for k in want:
                if want[k].dtype.is_floating_point:
                    torch.testing.assert_close(got[k], want[k], rtol=1e-4, atol=1e-6, equal_nan=True, msg=k)
                else:
                    assert torch.equal(got[k], want[k]), k


def test_noalloc_entry_point_refuses_requests_beyond_its_scratch():
    big = B.make_params(8192, 12, 152064, B.PPOW_BF16, B.PPOW_GREEDY, 0.03)
    assert B.ppow_score_workspace_bytes(big) > B.ppow_noalloc_scratch_bytes()
    dummy = torch.zeros(8, dtype=torch.bfloat16, device=DEV)
    tok = torch.zeros(8, dtype=torch.int32, device=DEV)
    out = {"accepted_len": torch.zeros(8, dtype=torch.int32, device=DEV)}
    with pytest.raises(B.PpowError) as e:                                     # refused before anything is launched
        B.ppow_score_windows_noalloc(big, dummy, dummy, tok, None, None, None, out)
    assert e.value.status == B.PPOW_ERR_UNSUPPORTED
    bad = B.make_params(4, 4, 1, B.PPOW_BF16, B.PPOW_GREEDY, 0.03)
    with pytest.raises(B.PpowError) as e:
        B.ppow_score_windows_noalloc(bad, dummy, dummy, tok, None, None, None, out)
    assert e.value.status == B.PPOW_ERR_INVALID_ARG
