"""GPU-vs-oracle parity through the C ABI on the five synthetic workloads and on edge cases."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2605_14978_b200 import binding as B
from paper_2605_14978_b200 import workloads as W

from parity_util import compare_scores, compare_selection, run_gpu, run_oracle

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

# (workload index, windows used for the element-by-element comparison)
SMALL = [(0, 64), (1, 96), (2, 48), (3, 80), (4, 24)]


def _check_workload(w, x, sample=None):
    reports = {}
    for mode in w.modes:
        gpu = run_gpu(x, mode, w.c, w.temperature)
        assert B.ppow_read_error_flags(gpu["_workspace"]) == 0
        ref = run_oracle(x, mode, w.c, w.temperature, windows=sample)
        rep = compare_scores(gpu, ref, mode, x["uniforms"], windows=sample)
        if sample is None:
            rep.update(compare_selection(gpu["score"], w.n_keep, ref["score"]))
        else:
            rep.update(compare_selection(gpu["score"], w.n_keep))
        # properties that hold at any size
        L = x["valid_len"] if x["valid_len"] is not None else torch.full((w.N,), w.K, device=DEV, dtype=torch.int32)
        assert bool(((gpu["accepted_len"] >= 0) & (gpu["accepted_len"] <= L)).all())
        assert bool((gpu["conf"] >= 0).all()) and bool((gpu["conf"] <= 1).all())
        assert bool((gpu["kl"] >= -1e-5).all())
        assert bool(torch.isfinite(gpu["score"]).all())
        # run-to-run determinism (catches races in the reductions)
        again = run_gpu(x, mode, w.c, w.temperature)
        for k, v in gpu.items():
            if not k.startswith("_"):
                assert torch.equal(v, again[k]), k
        reports[mode] = rep
    return reports


@pytest.mark.parametrize("idx,n", SMALL)
def test_workload_reduced_windows_elementwise(idx, n):
    w = W.scaled(W.WORKLOADS[idx], n)
    x = W.generate(w, DEV)
    rep = _check_workload(w, x)
    print(w.name, rep)


@pytest.mark.parametrize("idx", [1, 2, 3, 4])
def test_workload_full_size_sampled(idx):
    """Full-size launch (the configuration the benchmark times); the oracle checks sampled windows."""
    w = W.WORKLOADS[idx]
    x = W.generate(w, DEV)
    per = 16 if idx >= 3 else 32
    mid = (w.N // 2 // 64) * 64 + 7
    sample = np.r_[0:per, mid:mid + per, w.N - per:w.N]
    rep = _check_workload(w, x, sample=torch.from_numpy(sample).to(DEV))
    print(w.name, rep)


# ------------------------------------------------------------------------------------ edge cases


def _random_inputs(N, K, V, dtype, seed, sigma=0.7, scale=2.0):
    g = torch.Generator(device=DEV).manual_seed(seed)
    t = (torch.randn((N, K, V), generator=g, device=DEV) * scale)
    d = t + sigma * torch.randn((N, K, V), generator=g, device=DEV)
    x = {"target_logits": t.to(dtype), "draft_logits": d.to(dtype),
         "draft_tokens": torch.randint(0, V, (N, K), generator=g, device=DEV, dtype=torch.int32),
         "uniforms": torch.rand((N, K), generator=g, device=DEV), "valid_len": None}
    return x


def _both_modes(x, c=0.05, temperature=1.0, eta=1.0, eps=0.5, ref_logp=None):
    for mode in ("greedy", "stochastic"):
        gpu = run_gpu(x, mode, c, temperature, eta, eps, ref_logp)
        ref = run_oracle(x, mode, c, temperature, eta, eps, ref_logp)
        compare_scores(gpu, ref, mode, x["uniforms"], eps=eps)
    return gpu, ref


@pytest.mark.parametrize("N,K,V,dtype", [
    (5, 1, 8, torch.bfloat16),          # smallest vector row
    (3, 32, 64, torch.bfloat16),        # largest K
    (7, 3, 1001, torch.bfloat16),       # odd V: scalar path, rows not 16-byte aligned
    (7, 3, 1001, torch.float32),
    (2, 2, 2, torch.float32),           # smallest vocabulary
    (4, 5, 8 * 2333, torch.bfloat16),   # several tiles plus a ragged tail of units
    (1, 8, 128256, torch.bfloat16),     # few rows, large V: rows are split into segments
    (3, 4, 50000, torch.float32),       # f32 rows of whole 16-byte units: bulk-copy kernel, rows split into segments
    (6, 2, 4 * (3 * 512 + 77), torch.float32),   # f32, several tiles plus a ragged tail of units
    (40, 8, 32000, torch.float32),      # f32, one item per row
    (2, 3, 4, torch.float32),           # one f32 unit per row
    (5, 8, 32000, torch.float16),       # f16: bulk-copy kernel
    (4, 5, 8 * 2333, torch.float16),    # f16, ragged tail of units
    (7, 3, 1001, torch.float16),        # f16, scalar kernel
    (1, 8, 128256, torch.float16),      # f16, rows split into segments
    # rows of 4 KB or less in a call of a few MB take the one-launch kernel (the cases above with V <= 1001);
    # the same kinds of shape just past that limit reach the bulk-copy and the scalar kernels
    (5, 1, 2056, torch.bfloat16),       # bulk-copy kernel: two tiles and one unit
    (3, 32, 2064, torch.bfloat16),      # bulk-copy kernel, largest K
    (7, 3, 5001, torch.bfloat16),       # odd V: rows start inside 16-byte units (bulk-copy kernel, first and last unit masked)
    (7, 3, 3001, torch.float32),
    (7, 3, 5001, torch.float16),
    (5, 4, 50257, torch.bfloat16),      # a real odd vocabulary size: several items per row, every row at another offset
    (3, 2, 128 * 8 * 3 + 1, torch.bfloat16),   # one logit more than three whole tiles: the last item gets an extra unit
    (3, 2, 128 * 4 * 2 - 1, torch.float32),
    (2, 3, 1028, torch.float32),        # f32 bulk-copy kernel: two tiles and one unit
    (131, 4, 1000, torch.float32),      # one-launch kernel at its size limit (4 MiB of logits)
    (132, 4, 1000, torch.float32),      # the same rows just past the limit: bulk-copy kernel, one short item per row
])
def test_shapes_and_paths(N, K, V, dtype):
    x = _random_inputs(N, K, V, dtype, seed=N * 1000 + K * 10 + V % 7)
    _both_modes(x, temperature=0.9)


def test_ragged_lengths_including_empty_windows():
    N, K, V = 40, 10, 4096
    x = _random_inputs(N, K, V, torch.bfloat16, seed=5)
    x["valid_len"] = torch.randint(0, K + 1, (N,), device=DEV, dtype=torch.int32)
    x["valid_len"][:3] = 0
    x["valid_len"][3] = K
    # poison the masked positions: they must be neither read into results nor scored
    for n in range(N):
        L = int(x["valid_len"][n])
        x["draft_tokens"][n, L:] = -7
    gpu, ref = _both_modes(x, eps=20.0)
    assert B.ppow_read_error_flags(gpu["_workspace"]) == 0        # masked tokens are not looked at
    for name in list(B.POSITION_OUTPUTS) + list(B.WINDOW_OUTPUTS):
        assert float(gpu[name][:3].float().abs().sum()) == 0.0     # empty windows: all outputs 0


@pytest.mark.parametrize("V,off_t,off_d", [
    (512, 1, 1),        # one-launch kernel
    (4096, 1, 1),       # both tensors one logit off a 16-byte boundary: bulk-copy kernel on shifted rows
    (4096, 5, 5),
    (4099, 0, 0),       # aligned base, odd V: every row starts at another offset
    (4099, 3, 3),
    (4096, 1, 3),       # tensors at different offsets within a unit: scalar row kernel
    (4099, 0, 2),
])
def test_unaligned_rows_and_base_pointers(V, off_t, off_d):
    N, K = 3, 2
    x = _random_inputs(N, K, V, torch.bfloat16, seed=6 + V + off_t)
    for key, off in (("target_logits", off_t), ("draft_logits", off_d)):
        flat = torch.full((N * K * V + 16,), 9000.0, dtype=torch.bfloat16, device=DEV)   # huge values around the tensor:
        flat[off:off + N * K * V].copy_(x[key].flatten())                                # they must never be scored
        x[key] = flat[off:off + N * K * V].view(N, K, V)
        assert x[key].data_ptr() % 16 == (2 * off) % 16
    _both_modes(x)


def test_float16_workload_and_ties():
    w = dataclasses.replace(W.scaled(W.WORKLOADS[2], 24), dtype="f16")       # the headline recipe stored as f16
    x = W.generate(w, DEV)
    _check_workload(w, x)
    xt = _random_inputs(3, 2, 4096, torch.float16, seed=18)
    top = xt["target_logits"].float().amax(-1, keepdim=True) + 1.0
    xt["target_logits"][:, :, torch.tensor([4095, 9, 2048, 8], device=DEV)] = top.to(torch.float16)
    gpu, _ = _both_modes(xt)
    assert bool((gpu["target_argmax"] == 8).all())


def test_f32_unaligned_base_pointer_and_ties():
    N, K, V = 3, 2, 2048
    x = _random_inputs(N, K, V, torch.float32, seed=16)
    t = x["target_logits"]
    top = t.amax(-1, keepdim=True) + 1.0
    t[:, :, torch.tensor([2047, 5, 1024, 4], device=DEV)] = top      # exact ties: index 4 wins
    gpu, ref = _both_modes(x)
    assert bool((gpu["target_argmax"] == 4).all())
    for key in ("target_logits", "draft_logits"):
        flat = torch.empty(N * K * V + 1, dtype=torch.float32, device=DEV)
        flat[1:].copy_(x[key].flatten())
        x[key] = flat[1:].view(N, K, V)                              # 4-byte aligned only: scalar kernel
        assert x[key].data_ptr() % 16 != 0
    gpu2, _ = _both_modes(x)
    assert bool((gpu2["target_argmax"] == 4).all())


def test_argmax_ties_take_lowest_index():
    N, K, V = 4, 3, 4096
    x = _random_inputs(N, K, V, torch.bfloat16, seed=7)
    t = x["target_logits"]
    top = t.float().amax(-1, keepdim=True) + 1.0
    idx = torch.tensor([4095, 17, 2048, 16, 3000], device=DEV)
    t[:, :, idx] = top.to(torch.bfloat16)                          # five exact ties for the maximum
    x["draft_tokens"][:, 0] = 16
    x["draft_tokens"][:, 1] = 17
    gpu, ref = _both_modes(x)
    assert bool((gpu["target_argmax"] == 16).all())
    g = run_gpu(x, "greedy", 0.05)
    assert bool((g["accept_flag"][:, 0] == 1).all()) and bool((g["accept_flag"][:, 1] == 0).all())
    # -0.0 and +0.0 tie
    z = torch.full((1, 1, 64), -3.0, device=DEV, dtype=torch.bfloat16)
    z[0, 0, 40] = 0.0
    z[0, 0, 9] = -0.0
    xz = {"target_logits": z, "draft_logits": z.clone(), "draft_tokens": torch.tensor([[9]], device=DEV, dtype=torch.int32),
          "uniforms": torch.zeros((1, 1), device=DEV), "valid_len": None}
    gz, rz = _both_modes(xz)
    assert int(gz["target_argmax"][0, 0]) == 9 == int(rz["target_argmax"][0, 0])


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16, torch.float32])
def test_argmax_ties_at_the_first_and_last_logit_of_rows_that_start_inside_a_unit(dtype):
    # odd V: row r starts r * V logits into the tensor, at a different offset within a 16-byte unit each time; the
    # maximum sits at the row's very first and very last logit (and once in the middle), next to the neighbours' data
    N, K, V = 3, 3, 4099
    x = _random_inputs(N, K, V, dtype, seed=23)
    t = x["target_logits"]
    top = t.float().amax(dim=(0, 1, 2)) + 1.0                       # one value above every row's maximum
    t[:, :, V - 1] = top.to(dtype)
    t[:, 1:, 2000] = top.to(dtype)
    t[:, 2, 0] = top.to(dtype)
    gpu, ref = _both_modes(x)
    want = torch.tensor([V - 1, 2000, 0], device=DEV, dtype=torch.int32).expand(N, K)
    assert torch.equal(gpu["target_argmax"], want)
    x["draft_logits"] = x["target_logits"].clone()                   # and identical tensors still give exactly zero
    g = run_gpu(x, "stochastic", 0.04)
    assert float(g["kl"].abs().max()) == 0.0 and bool((g["accepted_len"] == K).all())


def test_identical_logits_zero_divergence_full_acceptance():
    x = _random_inputs(6, 8, 32000, torch.bfloat16, seed=8)
    x["draft_logits"] = x["target_logits"].clone()
    gpu = run_gpu(x, "stochastic", 0.04)
    assert float(gpu["kl"].abs().max()) == 0.0 and float(gpu["score"].abs().max()) == 0.0
    assert bool((gpu["accepted_len"] == 8).all())
    t = x["target_logits"].float()
    first_max = torch.where(t == t.amax(-1, keepdim=True), torch.arange(t.shape[-1], device=DEV), t.shape[-1]).amin(-1)
    x["draft_tokens"] = first_max.to(torch.int32)                  # lowest index among tied maxima
    gpu = run_gpu(x, "greedy", 0.04)
    assert bool((gpu["accepted_len"] == 8).all()) and float(gpu["delta"].abs().max()) == 0.0
    _both_modes(x)


def test_out_of_range_tokens_are_rejected_and_flagged():
    x = _random_inputs(4, 4, 800, torch.bfloat16, seed=9)
    x["draft_tokens"][1, 2] = 800
    x["draft_tokens"][2, 0] = -1
    gpu, ref = _both_modes(x)
    assert B.ppow_read_error_flags(gpu["_workspace"]) & B.PPOW_FLAG_TOKEN_RANGE
    assert int(gpu["accept_flag"][1, 2]) == 0 and int(gpu["accepted_len"][2]) == 0
    assert float(gpu["logp_tok"][1, 2]) == float("-inf")


def test_extreme_rows_exercise_reference_rebasing():
    N, K, V = 4, 4, 8 * 1024
    g = torch.Generator(device=DEV).manual_seed(10)
    # steadily rising rows: almost every tile raises the running reference by far more than 2^64
    ramp = torch.arange(V, device=DEV, dtype=torch.float32) * 0.9
    t = ramp.view(1, 1, V) + torch.randn((N, K, V), generator=g, device=DEV)
    d = ramp.flip(0).view(1, 1, V) * 0.5 + torch.randn((N, K, V), generator=g, device=DEV)
    x = {"target_logits": t.to(torch.bfloat16), "draft_logits": d.to(torch.bfloat16),
         "draft_tokens": torch.randint(0, V, (N, K), generator=g, device=DEV, dtype=torch.int32),
         "uniforms": torch.rand((N, K), generator=g, device=DEV), "valid_len": None}
    x["draft_tokens"][:, 0] = V - 1
    _both_modes(x)
    # Student-t spikes on both sides, float32 storage
    spikes = torch.distributions.StudentT(3.0).sample((N, K, V)).to(DEV) * 400.0
    x["target_logits"] = spikes.float()
    x["draft_logits"] = (spikes + torch.distributions.StudentT(3.0).sample((N, K, V)).to(DEV) * 200.0).float()
    _both_modes(x)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32, torch.float16])
@pytest.mark.parametrize("top", [12.0, 15.5, 16.5, 17.5])
def test_one_confident_token_over_a_flat_tail(top, dtype):
    """The hardest case for single-precision sums: one term decides the sum and 128255 equal terms, each
    near half an ulp of it, follow.  Every add after the big term rounds the same way, so the error grows
    with the number of adds between two compensated folds; this pins that interval."""
    N, K, V = 4, 8, 128256
    g = torch.Generator(device=DEV).manual_seed(int(top * 10))
    pos = torch.randint(0, V // 8, (N, K), generator=g, device=DEV) * 8      # first logit of a 16-byte unit
    t = torch.zeros((N, K, V), device=DEV).scatter_(2, pos[..., None], top).to(dtype)
    d = torch.zeros((N, K, V), device=DEV).scatter_(2, pos[..., None], top - 1.0).to(dtype)
    x = {"target_logits": t, "draft_logits": d, "draft_tokens": pos.to(torch.int32),
         "uniforms": torch.rand((N, K), generator=g, device=DEV), "valid_len": None}
    gpu, ref = _both_modes(x, c=0.04)
    assert bool((gpu["target_argmax"] == pos).all())


def test_reference_window_logprob_variant_of_delta():
    x = _random_inputs(9, 5, 2048, torch.bfloat16, seed=11, sigma=0.2)
    ref_logp = -torch.rand(9, device=DEV) * 3.0
    gpu, ref = _both_modes(x, eps=30.0, eta=0.7, ref_logp=ref_logp)
    assert float(gpu["reward_dist"].max()) in (0.0, pytest.approx(0.7))


def test_temperature_and_cost_parameters():
    x = _random_inputs(6, 6, 4000, torch.bfloat16, seed=12)
    for T, c in ((0.5, 0.0), (0.7, 0.12), (3.0, 1.5)):
        _both_modes(x, c=c, temperature=T)


def test_optional_outputs_may_be_omitted():
    x = _random_inputs(4, 4, 1024, torch.bfloat16, seed=13)
    p = B.make_params(4, 4, 1024, B.PPOW_BF16, B.PPOW_GREEDY, 0.05)
    ws = B.alloc_workspace(B.ppow_score_workspace_bytes(p), DEV)
    out = {"accepted_len": torch.full((4,), -1, device=DEV, dtype=torch.int32),
           "score": torch.zeros(4, device=DEV)}
    B.ppow_score_windows(p, x["draft_logits"], x["target_logits"], x["draft_tokens"], None, None, None, out, ws)
    torch.cuda.synchronize()
    full = run_gpu(x, "greedy", 0.05)
    assert torch.equal(out["accepted_len"], full["accepted_len"]) and torch.equal(out["score"], full["score"])


# ------------------------------------------------------------------------------------ selection


@pytest.mark.parametrize("N,n_keep", [(1, 1), (2, 1), (64, 16), (1000, 1000), (4096, 410), (8192, 1639), (16384, 3),
                                      (16385, 100), (70000, 14000), (3000, 0)])
def test_selection_bit_exact_with_ties(N, n_keep):
    g = torch.Generator(device=DEV).manual_seed(N + n_keep)
    s = torch.rand(N, generator=g, device=DEV)
    tie = torch.randint(0, N, (N // 3 + 1,), generator=g, device=DEV)
    s[tie] = 0.5                                                    # many exact ties, some at the cut
    s[torch.randint(0, N, (3,), generator=g, device=DEV)] = 0.0
    s[torch.randint(0, N, (3,), generator=g, device=DEV)] = -0.0
    compare_selection(s, n_keep)
    compare_selection(torch.full((N,), 2.5, device=DEV), n_keep)    # all equal: the first n_keep indices
    compare_selection(-s, n_keep)                                   # negative scores order correctly


def test_status_codes_for_bad_arguments():
    x = _random_inputs(2, 2, 64, torch.bfloat16, seed=14)
    p = B.make_params(2, 2, 64, B.PPOW_BF16, B.PPOW_STOCHASTIC, 0.05)
    ws = B.alloc_workspace(B.ppow_score_workspace_bytes(p), DEV)
    out = B.alloc_outputs(2, 2, DEV)

    def status(params=p, uniforms=x["uniforms"], outputs=out, workspace=ws):
        try:
            B.ppow_score_windows(params, x["draft_logits"], x["target_logits"], x["draft_tokens"], uniforms, None,
                                 None, outputs, workspace)
        except B.PpowError as e:
            return e.status
        return B.PPOW_OK

    assert status() == B.PPOW_OK
    assert status(uniforms=None) == B.PPOW_ERR_INVALID_ARG                      # stochastic needs uniforms
    assert status(params=B.make_params(2, 2, 64, B.PPOW_BF16, 1, 0.05, temperature=0.0)) == B.PPOW_ERR_INVALID_ARG
    assert status(params=B.make_params(2, 2, 1, B.PPOW_BF16, 1, 0.05)) == B.PPOW_ERR_INVALID_ARG
    assert status(params=B.make_params(2, 33, 64, B.PPOW_BF16, 1, 0.05)) == B.PPOW_ERR_UNSUPPORTED
    assert status(params=B.make_params(2, 2, 64, B.PPOW_BF16, 1, -1.0)) == B.PPOW_ERR_INVALID_ARG
    assert status(workspace=ws[:16]) == B.PPOW_ERR_WORKSPACE
    assert status(workspace=ws[1:]) == B.PPOW_ERR_WORKSPACE                     # misaligned
    assert status(outputs={}) == B.PPOW_ERR_INVALID_ARG                         # accepted_len is required
    assert status(params=B.make_params(0, 2, 64, B.PPOW_BF16, 1, 0.05)) == B.PPOW_OK   # N = 0: no-op
    torch.cuda.synchronize()
    s = torch.rand(10, device=DEV)
    with pytest.raises(B.PpowError):
        B.select_windows(s, 11)


@pytest.mark.parametrize("V", [4096, 5001])                          # rows of whole units / rows that start inside a unit
def test_host_buffer_entry_point_matches_device_path_with_chunking(V):
    w = W.scaled(W.WORKLOADS[3], 70)
    w = dataclasses.replace(w, V=V)
    x = W.generate(w, DEV)
    dev_out = run_gpu(x, "stochastic", w.c, w.temperature)
    dev_sel = B.select_windows(dev_out["score"], w.n_keep)
    params = B.make_params(w.N, w.K, w.V, B.PPOW_BF16, B.PPOW_STOCHASTIC, w.c, w.temperature)
    host = {k: (None if v is None else v.cpu().pin_memory()) for k, v in x.items()}
    for chunk in (w.N, 16, 1):                                       # one chunk, several, one window at a time
        out_host = {k: torch.zeros(v.shape, dtype=v.dtype).pin_memory() for k, v in dev_out.items() if not k.startswith("_")}
        sel_host = torch.zeros((w.n_keep,), dtype=torch.int32).pin_memory()
        mask_host = torch.zeros((w.N,), dtype=torch.uint8).pin_memory()
        scratch = B.alloc_workspace(B.ppow_host_scratch_bytes(params, chunk), DEV)
        B.ppow_score_and_select_host(params, host["draft_logits"], host["target_logits"], host["draft_tokens"],
                                     host["uniforms"], host["valid_len"], None, out_host, w.n_keep, sel_host, mask_host,
                                     scratch)
        torch.cuda.synchronize()
        for k, v in out_host.items():
            if V % 8 == 0 or not v.dtype.is_floating_point:      # whole units: the same lanes add the same logits
                assert torch.equal(v, dev_out[k].cpu()), (chunk, k)
            else:                                                # rows start at other offsets in a staged chunk than in
                torch.testing.assert_close(v, dev_out[k].cpu(), rtol=1e-5, atol=1e-6, msg=str((chunk, k)))   # the batch
        if V % 8 == 0:
            assert torch.equal(sel_host, dev_sel.cpu())
        else:
            want = oracle.select_windows(out_host["score"].numpy().astype(np.float64), w.n_keep)
            np.testing.assert_array_equal(sel_host.numpy(), want)
        assert int(mask_host.sum()) == w.n_keep
    with pytest.raises(B.PpowError):
        B.ppow_score_and_select_host(params, host["draft_logits"], host["target_logits"], host["draft_tokens"],
                                     host["uniforms"], host["valid_len"], None, out_host, w.n_keep, sel_host, None,
                                     B.alloc_workspace(1024, DEV))


def test_host_buffer_entry_point_with_a_shorter_last_chunk_at_full_vocabulary_width():
    # 477 windows staged as 296 + 181 at V = 32000: the two chunks and the whole batch are cut into work items
    # three different ways, and the scratch size the library asks for has to serve both chunk sizes
    w = W.scaled(W.WORKLOADS[1], 477)
    chunk = 296
    x = W.generate(w, DEV)
    dev_out = run_gpu(x, "greedy", w.c, w.temperature)
    dev_sel = B.select_windows(dev_out["score"], w.n_keep)
    torch.cuda.synchronize()
    params = B.make_params(w.N, w.K, w.V, B.PPOW_BF16, B.PPOW_GREEDY, w.c, w.temperature)
    host = {k: (None if v is None else v.cpu()) for k, v in x.items()}
    out_host = {k: torch.zeros(v.shape, dtype=v.dtype) for k, v in dev_out.items() if not k.startswith("_")}
    sel_host = torch.zeros((w.n_keep,), dtype=torch.int32)
    scratch = B.alloc_workspace(B.ppow_host_scratch_bytes(params, chunk), DEV)
    B.ppow_score_and_select_host(params, host["draft_logits"], host["target_logits"], host["draft_tokens"],
                                 None, None, None, out_host, w.n_keep, sel_host, None, scratch)
    torch.cuda.synchronize()
    for k, v in out_host.items():                                    # the chunks are cut into other work items than
        if v.dtype.is_floating_point:                                # the whole batch: floats agree to rounding
            torch.testing.assert_close(v, dev_out[k].cpu(), rtol=1e-5, atol=1e-6, msg=k)
        else:
            assert torch.equal(v, dev_out[k].cpu()), k
    want = oracle.select_windows(out_host["score"].numpy().astype(np.float64), w.n_keep)
    np.testing.assert_array_equal(sel_host.numpy(), want)
    assert len(set(sel_host.tolist()) ^ set(dev_sel.cpu().tolist())) <= 2


@pytest.mark.parametrize("T,scale", [(0.7, 8.0), (1.7, 8.0), (0.7, 2.0)])
def test_uniforms_just_outside_the_band_around_alpha(T, scale):
    """The kernel scales logits by log2(e)/T rounded to float32, i.e. it evaluates the softmax at T(1 + e) with
    |e| <= 2^-24; the shift of log alpha is e * (log alpha + H(P) - H(Q)).  Stress: wide logits, T != 1, drafted
    tokens chosen so that alpha is mid-range -- once the likeliest such token, once the least likely one (90 nats
    below the mode at scale 8) -- and uniforms placed 1.5e-6 on either side of the oracle's alpha, just outside
    the band in which flags may differ: every flag must equal the oracle's."""
    N, K, V = 8, 8, 32000
    x = _random_inputs(N, K, V, torch.bfloat16, seed=int(10 * T + scale), sigma=1.0, scale=scale)
    lp = torch.log_softmax(x["target_logits"].double() / T, -1)
    lq = torch.log_softmax(x["draft_logits"].double() / T, -1)
    mid = ((lp - lq).exp() > 0.2) & ((lp - lq).exp() < 0.8)
    picks = {"likely": torch.where(mid, lp, torch.full_like(lp, -1e9)).argmax(-1),
             "unlikely": torch.where(mid, lp, torch.full_like(lp, 1e9)).argmin(-1)}
    for name, tok in picks.items():
        x["draft_tokens"] = tok.to(torch.int32)
        x["uniforms"] = torch.zeros((N, K), device=DEV)
        alpha = run_oracle(x, "stochastic", 0.05, T)["alpha"]
        assert 0.2 < alpha.min() and alpha.max() < 0.8
        for side in (+1.0, -1.0):
            u = (alpha + side * 1.5e-6).astype(np.float32)
            x["uniforms"] = torch.from_numpy(u).to(DEV)
            gpu = run_gpu(x, "stochastic", 0.05, T)
            ref = run_oracle(x, "stochastic", 0.05, T)
            rep = compare_scores(gpu, ref, "stochastic", x["uniforms"])
            assert rep["band_flag_differences"] == 0, (name, side, rep)
            assert (ref["accept_flag"] == (side < 0)).all()          # the uniforms sit where they were meant to


def test_randomised_shapes_parameters_and_masks():
    """Property-style sweep: seeded random shapes (odd and even V, one position to 32, one window to dozens),
    storage types, temperatures, costs, ragged masks, logit scales and base-pointer offsets; everything is compared
    with the oracle."""
    rng = np.random.default_rng(2024)
    for case in range(60):
        N = int(rng.integers(1, 40))
        K = int(rng.choice([1, 2, 3, 5, 8, 10, 12, 17, 32]))
        V = int(rng.choice([2, 3, 8, 9, 64, 257, 1000, 1024, 2049, 4096 + 8, 5000, 5001, 20000, 40004, 50257]))
        if N * K * V > 6_000_000:
            N = max(1, 6_000_000 // (K * V))
        dtype = [torch.bfloat16, torch.float32, torch.float16][int(rng.choice(3, p=[0.5, 0.25, 0.25]))]
        T = float(rng.choice([0.5, 0.7, 1.0, 1.7]))
        c = float(rng.choice([0.0, 0.03, 0.12, 0.5]))
        scale = float(rng.choice([0.3, 2.0, 8.0]))
        x = _random_inputs(N, K, V, dtype, seed=1000 + case, sigma=float(rng.choice([0.0, 0.3, 1.5])), scale=scale)
        off_t = int(rng.choice([0, 0, 1, 3]))                       # base pointers off a 16-byte boundary, mostly by the
        off_d = off_t if rng.random() < 0.8 else int(rng.choice([0, 2]))   # same amount (else: the scalar row kernel)
        if off_t or off_d:
            for key, off in (("target_logits", off_t), ("draft_logits", off_d)):
                flat = torch.full((N * K * V + 16,), 100.0, dtype=dtype, device=DEV)
                flat[off:off + N * K * V].copy_(x[key].flatten())
                x[key] = flat[off:off + N * K * V].view(N, K, V)
        if rng.random() < 0.5:
            x["valid_len"] = torch.from_numpy(rng.integers(0, K + 1, size=N).astype(np.int32)).to(DEV)
        if rng.random() < 0.3:                                       # drafted tokens that are the target's choice
            t = x["target_logits"].float()
            x["draft_tokens"] = torch.where(t == t.amax(-1, keepdim=True), torch.arange(V, device=DEV), V).amin(-1).to(torch.int32)
        try:
            _both_modes(x, c=c, temperature=T, eta=float(rng.choice([1.0, 0.4])), eps=float(rng.choice([0.5, 3.0])))
        except AssertionError as e:
            raise AssertionError("case %d: N=%d K=%d V=%d %s T=%g c=%g scale=%g: %s" % (case, N, K, V, dtype, T, c, scale, e))


def test_bounded_device_wait_reports_a_timeout_and_leaves_the_context_usable():
    """Failure detection on the device: the copy pipeline's waits are bounded and report through the error
    word.  The self-test makes such a wait run out (an mbarrier nothing completes) without faulting anything."""
    ws = B.alloc_workspace(4096, DEV)
    B.ppow_selftest_wait_timeout(ws, probes=32)
    status, flags = B.ppow_read_error_status(ws)
    assert status == B.PPOW_ERR_DEVICE_TIMEOUT and flags & B.PPOW_FLAG_DEVICE_TIMEOUT
    assert "timeout" in B.ppow_status_string(status).lower() or "wait" in B.ppow_status_string(status).lower()
    # the context is intact: an ordinary scoring call on the same workspace works and clears the word
    x = _random_inputs(4, 4, 4096, torch.bfloat16, seed=31)
    gpu, _ = _both_modes(x)
    assert B.ppow_read_error_status(gpu["_workspace"]) == (B.PPOW_OK, 0)
    with pytest.raises(B.PpowError):
        B.ppow_selftest_wait_timeout(ws, probes=0)
    with pytest.raises(B.PpowError):
        B.ppow_selftest_wait_timeout(ws[1:], probes=8)
