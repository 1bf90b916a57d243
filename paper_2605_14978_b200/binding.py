"""ctypes binding of ``libppow.so``: the same entry points as ``include/ppow.h``, marshalling only.

Every step of the scoring path runs in the CUDA library.  There is no CPU or PyTorch fallback: if
the library has not been built, or a tensor is not on a CUDA device, the call raises.
PyTorch is used for device memory and streams only.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# PPOW_LIBRARY=checked loads the bounds-checked build of the same sources (see ppow_checked_failures)
#                        timeline loads the build whose row kernel records a per-warp timeline (ppow_timeline_read)
LIB_PATH = os.path.join(_HERE, {"checked": "libppow_checked.so", "timeline": "libppow_timeline.so"}.get(
    os.environ.get("PPOW_LIBRARY", ""), "libppow.so"))

PPOW_OK = 0
PPOW_ERR_INVALID_ARG, PPOW_ERR_UNSUPPORTED, PPOW_ERR_WORKSPACE, PPOW_ERR_CUDA, PPOW_ERR_DEVICE_TIMEOUT = 1, 2, 3, 4, 5
PPOW_GREEDY, PPOW_STOCHASTIC = 0, 1
PPOW_F32, PPOW_BF16, PPOW_F16 = 0, 1, 2
LOGIT_DTYPES = {PPOW_F32: torch.float32, PPOW_BF16: torch.bfloat16, PPOW_F16: torch.float16}
DTYPE_CODES = {v: k for k, v in LOGIT_DTYPES.items()}
PPOW_FLAG_TOKEN_RANGE, PPOW_FLAG_DEVICE_TIMEOUT, PPOW_FLAG_BOUNDS = 1, 2, 4

EXPORTS = ("ppow_score_workspace_bytes", "ppow_score_windows", "ppow_score_windows_traced", "ppow_read_error_flags",
           "ppow_select_workspace_bytes", "ppow_select_windows", "ppow_host_scratch_bytes",
           "ppow_score_and_select_host", "ppow_noalloc_scratch_bytes", "ppow_score_windows_noalloc",
           "ppow_noalloc_read_error_flags",
           "ppow_group_advantage", "ppow_sequence_windows", "ppow_sequence_windows_mixed", "ppow_expected_acceptance",
           "ppow_reference_logprob", "ppow_selftest_wait_timeout", "ppow_stream_read_probe", "ppow_score_kernel_launches",
           "ppow_checked_failures", "ppow_timeline_read", "ppow_status_string", "ppow_version")

POSITION_OUTPUTS = {"accept_flag": torch.uint8, "kl": torch.float32, "conf": torch.float32, "crit": torch.float32,
                    "logp_tok": torch.float32, "logq_tok": torch.float32, "target_argmax": torch.int32}
WINDOW_OUTPUTS = {"accepted_len": torch.int32, "reward_speedup": torch.float32, "reward_dist": torch.float32,
                  "reward": torch.float32, "delta": torch.float32, "score": torch.float32}
# training-side outputs of the scoring pass, written only when asked for
TRAIN_POSITION_OUTPUTS = {"kl_rev": torch.float32, "nabla": torch.float32, "lse_p": torch.float32,
                          "lse_q": torch.float32}
TRAIN_WINDOW_OUTPUTS = {"kl_rev_mean": torch.float32}
_ALL_OUTPUTS = {**POSITION_OUTPUTS, **WINDOW_OUTPUTS, **TRAIN_POSITION_OUTPUTS, **TRAIN_WINDOW_OUTPUTS}


class ppow_params(ctypes.Structure):
    _fields_ = [("N", ctypes.c_int32), ("K", ctypes.c_int32), ("V", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("mode", ctypes.c_int32),
                ("c", ctypes.c_float), ("temperature", ctypes.c_float),
                ("eta", ctypes.c_float), ("eps", ctypes.c_float)]


class ppow_outputs(ctypes.Structure):
    # field order is the order of the C struct
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("accept_flag", "accepted_len", "reward_speedup", "reward_dist", "reward", "delta", "score",
                 "kl", "conf", "crit", "logp_tok", "logq_tok", "target_argmax",
                 "kl_rev", "kl_rev_mean", "nabla", "lse_p", "lse_q")]


class PpowError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s (status %d)" % (where, ppow_status_string(status), status))


_lib = None


def load_library():
    """Load libppow.so; raises if it was not built (there is no fallback path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("libppow.so is missing: build it with `python -m paper_2605_14978_b200.build` "
                           "(the scoring path has no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    lib.ppow_score_workspace_bytes.restype = sz
    lib.ppow_score_workspace_bytes.argtypes = [ctypes.POINTER(ppow_params)]
    lib.ppow_score_windows.restype = ctypes.c_int
    lib.ppow_score_windows.argtypes = [ctypes.POINTER(ppow_params), vp, vp, vp, vp, vp, vp,
                                       ctypes.POINTER(ppow_outputs), vp, sz, vp]
    lib.ppow_score_windows_traced.restype = ctypes.c_int
    lib.ppow_score_windows_traced.argtypes = lib.ppow_score_windows.argtypes + [vp, vp]
    lib.ppow_read_error_flags.restype = ctypes.c_int
    lib.ppow_read_error_flags.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32), vp]
    lib.ppow_select_workspace_bytes.restype = sz
    lib.ppow_select_workspace_bytes.argtypes = [i32]
    lib.ppow_select_windows.restype = ctypes.c_int
    lib.ppow_select_windows.argtypes = [vp, i32, i32, vp, vp, vp, sz, vp]
    lib.ppow_host_scratch_bytes.restype = sz
    lib.ppow_host_scratch_bytes.argtypes = [ctypes.POINTER(ppow_params), i32]
    lib.ppow_score_and_select_host.restype = ctypes.c_int
    lib.ppow_score_and_select_host.argtypes = [ctypes.POINTER(ppow_params), vp, vp, vp, vp, vp, vp,
                                               ctypes.POINTER(ppow_outputs), i32, vp, vp, vp, sz, vp]
    lib.ppow_noalloc_scratch_bytes.restype = sz
    lib.ppow_noalloc_scratch_bytes.argtypes = []
    lib.ppow_score_windows_noalloc.restype = ctypes.c_int
    lib.ppow_score_windows_noalloc.argtypes = [ctypes.POINTER(ppow_params), vp, vp, vp, vp, vp, vp,
                                               ctypes.POINTER(ppow_outputs), vp]
    lib.ppow_noalloc_read_error_flags.restype = ctypes.c_int
    lib.ppow_noalloc_read_error_flags.argtypes = [ctypes.POINTER(ctypes.c_uint32), vp]
    lib.ppow_group_advantage.restype = ctypes.c_int
    lib.ppow_group_advantage.argtypes = [vp, i32, i32, ctypes.c_float, vp, vp]
    lib.ppow_sequence_windows.restype = ctypes.c_int
    lib.ppow_sequence_windows.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp]
    lib.ppow_sequence_windows_mixed.restype = ctypes.c_int
    lib.ppow_sequence_windows_mixed.argtypes = [vp, vp, i32, i32, ctypes.c_float, vp, vp, vp, vp, vp]
    lib.ppow_expected_acceptance.restype = ctypes.c_int
    lib.ppow_expected_acceptance.argtypes = [ctypes.POINTER(ppow_params), vp, vp, vp, vp, vp, vp, vp]
    lib.ppow_reference_logprob.restype = ctypes.c_int
    lib.ppow_reference_logprob.argtypes = [ctypes.POINTER(ppow_params), vp, vp, vp, vp, vp]
    lib.ppow_selftest_wait_timeout.restype = ctypes.c_int
    lib.ppow_selftest_wait_timeout.argtypes = [vp, sz, ctypes.c_uint32, vp]
    lib.ppow_stream_read_probe.restype = ctypes.c_int
    lib.ppow_stream_read_probe.argtypes = [vp, sz, vp, vp]
    lib.ppow_score_kernel_launches.restype = ctypes.c_int
    lib.ppow_score_kernel_launches.argtypes = [ctypes.POINTER(ppow_params)]
    lib.ppow_checked_failures.restype = ctypes.c_int
    lib.ppow_checked_failures.argtypes = [ctypes.POINTER(ctypes.c_uint32), ctypes.POINTER(ctypes.c_uint32)]
    lib.ppow_timeline_read.restype = ctypes.c_int
    lib.ppow_timeline_read.argtypes = [vp, sz]
    lib.ppow_status_string.restype = ctypes.c_char_p
    lib.ppow_status_string.argtypes = [ctypes.c_int]
    lib.ppow_version.restype = ctypes.c_int
    lib.ppow_version.argtypes = []
    _lib = lib
    return lib


def ppow_status_string(status: int) -> str:
    return load_library().ppow_status_string(int(status)).decode()


def ppow_version() -> int:
    return int(load_library().ppow_version())


def _dev_ptr(t: Optional[torch.Tensor], dtype=None, name="tensor"):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("%s must live on a CUDA device (no CPU path exists)" % name)
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    if dtype is not None and t.dtype != dtype:
        raise ValueError("%s must have dtype %s, got %s" % (name, dtype, t.dtype))
    return ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def make_params(N, K, V, dtype, mode, c, temperature=1.0, eta=1.0, eps=0.5) -> ppow_params:
    return ppow_params(int(N), int(K), int(V), int(dtype), int(mode), float(c), float(temperature),
                       float(eta), float(eps))


def ppow_score_workspace_bytes(params: ppow_params) -> int:
    return int(load_library().ppow_score_workspace_bytes(ctypes.byref(params)))


def ppow_score_kernel_launches(params: ppow_params) -> int:
    return int(load_library().ppow_score_kernel_launches(ctypes.byref(params)))


def ppow_stream_read_probe(data: torch.Tensor, checksum: torch.Tensor, stream=None) -> None:
    """One read-only streaming pass over ``data`` (any dtype, contiguous, a multiple of 16 bytes); XOR of its
    32-bit words into ``checksum`` (one int32/uint32-sized CUDA element)."""
    lib = load_library()
    st = lib.ppow_stream_read_probe(_dev_ptr(data, None, "data"), data.numel() * data.element_size(),
                                    _dev_ptr(checksum, None, "checksum"), _stream_ptr(stream))
    if st != PPOW_OK:
        raise PpowError(st, "ppow_stream_read_probe")


def ppow_checked_failures():
    """(status, failed checks, first failing site) of the bounds-checked build; status PPOW_ERR_UNSUPPORTED and
    zeros from the ordinary library."""
    f, site = ctypes.c_uint32(0), ctypes.c_uint32(0)
    st = load_library().ppow_checked_failures(ctypes.byref(f), ctypes.byref(site))
    return int(st), int(f.value), int(site.value)


def ppow_timeline_read(warps: int):
    """(status, array [warps, 11] of uint64) from the timeline build; status PPOW_ERR_UNSUPPORTED otherwise."""
    import numpy as np
    buf = np.zeros((int(warps), 11), dtype=np.uint64)
    st = load_library().ppow_timeline_read(ctypes.c_void_p(buf.ctypes.data), int(warps))
    return int(st), buf


def ppow_select_workspace_bytes(N: int) -> int:
    return int(load_library().ppow_select_workspace_bytes(int(N)))


def alloc_outputs(N: int, K: int, device) -> dict:
    out = {k: torch.empty((N, K), dtype=dt, device=device) for k, dt in POSITION_OUTPUTS.items()}
    out.update({k: torch.empty((N,), dtype=dt, device=device) for k, dt in WINDOW_OUTPUTS.items()})
    return out


def alloc_train_outputs(N: int, K: int, device) -> dict:
    out = {k: torch.empty((N, K), dtype=dt, device=device) for k, dt in TRAIN_POSITION_OUTPUTS.items()}
    out.update({k: torch.empty((N,), dtype=dt, device=device) for k, dt in TRAIN_WINDOW_OUTPUTS.items()})
    return out


def alloc_workspace(nbytes: int, device) -> torch.Tensor:
    # torch's caching allocator returns 512-byte aligned blocks
    return torch.empty((max(int(nbytes), 256),), dtype=torch.uint8, device=device)


def _event_ptr(ev):
    """cudaEvent_t of a torch.cuda.Event (created on first record), or NULL."""
    if ev is None:
        return None
    if not ev.cuda_event:
        ev.record()           # torch creates the CUDA event lazily; the library re-records it
    return ctypes.c_void_p(ev.cuda_event)


def ppow_score_windows(params: ppow_params, draft_logits, target_logits, draft_tokens, uniforms, valid_len,
                       ref_logp, outputs: dict, workspace: torch.Tensor, stream=None) -> None:
    """Enqueue the scoring pass; raises PpowError on a non-OK status.  ``outputs`` maps output names
    to preallocated CUDA tensors (absent or None = not written; ``accepted_len`` is required)."""
    ppow_score_windows_traced(params, draft_logits, target_logits, draft_tokens, uniforms, valid_len, ref_logp,
                              outputs, workspace, stream, None, None)


def ppow_score_windows_traced(params: ppow_params, draft_logits, target_logits, draft_tokens, uniforms, valid_len,
                              ref_logp, outputs: dict, workspace: torch.Tensor, stream=None,
                              event_reduce_begin=None, event_reduce_end=None) -> None:
    """ppow_score_windows plus two optional torch.cuda.Event objects recorded around the row-reduction kernel."""
    lib = load_library()
    lt = LOGIT_DTYPES[params.dtype]
    o = ppow_outputs()
    for name, _ in ppow_outputs._fields_:
        t = outputs.get(name)
        want = _ALL_OUTPUTS[name]
        p = _dev_ptr(t, want, name)
        setattr(o, name, p.value if p is not None else None)
    traced = event_reduce_begin is not None or event_reduce_end is not None
    fn = lib.ppow_score_windows_traced if traced else lib.ppow_score_windows
    extra = (_event_ptr(event_reduce_begin), _event_ptr(event_reduce_end)) if traced else ()
    st = fn(
        ctypes.byref(params),
        _dev_ptr(draft_logits, lt, "draft_logits"), _dev_ptr(target_logits, lt, "target_logits"),
        _dev_ptr(draft_tokens, torch.int32, "draft_tokens"), _dev_ptr(uniforms, torch.float32, "uniforms"),
        _dev_ptr(valid_len, torch.int32, "valid_len"), _dev_ptr(ref_logp, torch.float32, "ref_logp"),
        ctypes.byref(o), _dev_ptr(workspace, torch.uint8, "workspace"),
        workspace.numel() if workspace is not None else 0, _stream_ptr(stream), *extra)
    if st != PPOW_OK:
        raise PpowError(st, "ppow_score_windows")


class ScoreCall:
    """The arguments of ``ppow_score_windows`` marshalled once.  ``launch()`` repeats the foreign call without
    rebuilding them, which matters when the same buffers are scored step after step and the problem is small
    enough for argument marshalling to show.  Holds references to the tensors; nothing is computed here."""

    def __init__(self, params: ppow_params, draft_logits, target_logits, draft_tokens, uniforms, valid_len, ref_logp,
                 outputs: dict, workspace: torch.Tensor):
        self._lib = load_library()
        lt = LOGIT_DTYPES[params.dtype]
        self._keep = (params, draft_logits, target_logits, draft_tokens, uniforms, valid_len, ref_logp, outputs, workspace)
        self._out = ppow_outputs()
        for name, _ in ppow_outputs._fields_:
            ptr = _dev_ptr(outputs.get(name), _ALL_OUTPUTS[name], name)
            setattr(self._out, name, ptr.value if ptr is not None else None)
        self._args = (ctypes.byref(params),
                      _dev_ptr(draft_logits, lt, "draft_logits"), _dev_ptr(target_logits, lt, "target_logits"),
                      _dev_ptr(draft_tokens, torch.int32, "draft_tokens"), _dev_ptr(uniforms, torch.float32, "uniforms"),
                      _dev_ptr(valid_len, torch.int32, "valid_len"), _dev_ptr(ref_logp, torch.float32, "ref_logp"),
                      ctypes.byref(self._out), _dev_ptr(workspace, torch.uint8, "workspace"),
                      workspace.numel() if workspace is not None else 0)

    def launch(self, stream=None, event_reduce_begin=None, event_reduce_end=None) -> None:
        if event_reduce_begin is None and event_reduce_end is None:
            st = self._lib.ppow_score_windows(*self._args, _stream_ptr(stream))
        else:
            st = self._lib.ppow_score_windows_traced(*self._args, _stream_ptr(stream), _event_ptr(event_reduce_begin),
                                                     _event_ptr(event_reduce_end))
        if st != PPOW_OK:
            raise PpowError(st, "ppow_score_windows")


class SelectCall:
    """The arguments of ``ppow_select_windows`` marshalled once (see ScoreCall)."""

    def __init__(self, score, n_keep: int, selected, mask, workspace):
        self._lib = load_library()
        self._keep = (score, selected, mask, workspace)
        self._args = (_dev_ptr(score, torch.float32, "score"), int(score.numel()) if score is not None else 0, int(n_keep),
                      _dev_ptr(selected, torch.int32, "selected"), _dev_ptr(mask, torch.uint8, "mask"),
                      _dev_ptr(workspace, torch.uint8, "workspace"), workspace.numel() if workspace is not None else 0)

    def launch(self, stream=None) -> None:
        st = self._lib.ppow_select_windows(*self._args, _stream_ptr(stream))
        if st != PPOW_OK:
            raise PpowError(st, "ppow_select_windows")


def ppow_read_error_flags(workspace: torch.Tensor, stream=None) -> int:
    lib = load_library()
    flags = ctypes.c_uint32(0)
    st = lib.ppow_read_error_flags(_dev_ptr(workspace, torch.uint8, "workspace"), ctypes.byref(flags),
                                   _stream_ptr(stream))
    if st not in (PPOW_OK, PPOW_ERR_DEVICE_TIMEOUT):
        raise PpowError(st, "ppow_read_error_flags")
    return int(flags.value)


def ppow_selftest_wait_timeout(workspace: torch.Tensor, probes: int = 64, stream=None) -> None:
    """Makes the bounded device-side wait run out on purpose (harmlessly); see include/ppow.h."""
    lib = load_library()
    st = lib.ppow_selftest_wait_timeout(_dev_ptr(workspace, torch.uint8, "workspace"), workspace.numel(), int(probes),
                                        _stream_ptr(stream))
    if st != PPOW_OK:
        raise PpowError(st, "ppow_selftest_wait_timeout")


def ppow_read_error_status(workspace: torch.Tensor, stream=None):
    """(status, flags) of ppow_read_error_flags without raising on PPOW_ERR_DEVICE_TIMEOUT."""
    lib = load_library()
    flags = ctypes.c_uint32(0)
    st = lib.ppow_read_error_flags(_dev_ptr(workspace, torch.uint8, "workspace"), ctypes.byref(flags), _stream_ptr(stream))
    return int(st), int(flags.value)


def ppow_select_windows(score, n_keep: int, selected, mask, workspace, stream=None) -> None:
    lib = load_library()
    N = int(score.numel()) if score is not None else 0
    st = lib.ppow_select_windows(
        _dev_ptr(score, torch.float32, "score"), N, int(n_keep), _dev_ptr(selected, torch.int32, "selected"),
        _dev_ptr(mask, torch.uint8, "mask"), _dev_ptr(workspace, torch.uint8, "workspace"),
        workspace.numel() if workspace is not None else 0, _stream_ptr(stream))
    if st != PPOW_OK:
        raise PpowError(st, "ppow_select_windows")


def ppow_noalloc_scratch_bytes() -> int:
    return int(load_library().ppow_noalloc_scratch_bytes())


def ppow_score_windows_noalloc(params: ppow_params, draft_logits, target_logits, draft_tokens, uniforms, valid_len,
                               ref_logp, outputs: dict, stream=None) -> None:
    """ppow_score_windows for callers that cannot hand over a workspace: the library's built-in 4 MiB
    scratch array is used instead.  The binding itself allocates nothing here; ``outputs`` must hold
    preallocated CUDA tensors.  Calls on one device must not overlap (they share the array)."""
    lib = load_library()
    lt = LOGIT_DTYPES[params.dtype]
    o = ppow_outputs()
    for name, _ in ppow_outputs._fields_:
        want = _ALL_OUTPUTS[name]
        p = _dev_ptr(outputs.get(name), want, name)
        setattr(o, name, p.value if p is not None else None)
    st = lib.ppow_score_windows_noalloc(
        ctypes.byref(params),
        _dev_ptr(draft_logits, lt, "draft_logits"), _dev_ptr(target_logits, lt, "target_logits"),
        _dev_ptr(draft_tokens, torch.int32, "draft_tokens"), _dev_ptr(uniforms, torch.float32, "uniforms"),
        _dev_ptr(valid_len, torch.int32, "valid_len"), _dev_ptr(ref_logp, torch.float32, "ref_logp"),
        ctypes.byref(o), _stream_ptr(stream))
    if st != PPOW_OK:
        raise PpowError(st, "ppow_score_windows_noalloc")


def ppow_noalloc_read_error_flags(stream=None):
    """(status, flags) left by the last ppow_score_windows_noalloc call on the current device."""
    flags = ctypes.c_uint32(0)
    st = load_library().ppow_noalloc_read_error_flags(ctypes.byref(flags), _stream_ptr(stream))
    return int(st), int(flags.value)


def ppow_group_advantage(reward, group_size: int, delta: float, advantage, stream=None) -> None:
    lib = load_library()
    N = int(reward.numel()) if reward is not None else 0
    st = lib.ppow_group_advantage(_dev_ptr(reward, torch.float32, "reward"), N, int(group_size), float(delta),
                                  _dev_ptr(advantage, torch.float32, "advantage"), _stream_ptr(stream))
    if st != PPOW_OK:
        raise PpowError(st, "ppow_group_advantage")


def ppow_sequence_windows(crit, seq_offsets, K: int, scores, uniforms, starts, stream=None) -> None:
    lib = load_library()
    B = int(seq_offsets.numel()) - 1 if seq_offsets is not None else 0
    st = lib.ppow_sequence_windows(_dev_ptr(crit, torch.float32, "crit"), _dev_ptr(seq_offsets, torch.int32, "seq_offsets"),
                                   B, int(K), _dev_ptr(scores, torch.float32, "scores"),
                                   _dev_ptr(uniforms, torch.float32, "uniforms"), _dev_ptr(starts, torch.int32, "starts"),
                                   _stream_ptr(stream))
    if st != PPOW_OK:
        raise PpowError(st, "ppow_sequence_windows")


def ppow_sequence_windows_mixed(crit, seq_offsets, K: int, hard_frac: float, scores, uniforms_mix, uniforms_draw,
                                starts, stream=None) -> None:
    lib = load_library()
    B = int(seq_offsets.numel()) - 1 if seq_offsets is not None else 0
    st = lib.ppow_sequence_windows_mixed(
        _dev_ptr(crit, torch.float32, "crit"), _dev_ptr(seq_offsets, torch.int32, "seq_offsets"), B, int(K),
        float(hard_frac), _dev_ptr(scores, torch.float32, "scores"), _dev_ptr(uniforms_mix, torch.float32, "uniforms_mix"),
        _dev_ptr(uniforms_draw, torch.float32, "uniforms_draw"), _dev_ptr(starts, torch.int32, "starts"),
        _stream_ptr(stream))
    if st != PPOW_OK:
        raise PpowError(st, "ppow_sequence_windows_mixed")


def ppow_expected_acceptance(params: ppow_params, draft_logits, target_logits, valid_len, lse_p, lse_q,
                             expected_accept, stream=None) -> None:
    lib = load_library()
    lt = LOGIT_DTYPES[params.dtype]
    st = lib.ppow_expected_acceptance(
        ctypes.byref(params), _dev_ptr(draft_logits, lt, "draft_logits"), _dev_ptr(target_logits, lt, "target_logits"),
        _dev_ptr(valid_len, torch.int32, "valid_len"), _dev_ptr(lse_p, torch.float32, "lse_p"),
        _dev_ptr(lse_q, torch.float32, "lse_q"), _dev_ptr(expected_accept, torch.float32, "expected_accept"),
        _stream_ptr(stream))
    if st != PPOW_OK:
        raise PpowError(st, "ppow_expected_acceptance")


def ppow_reference_logprob(params: ppow_params, ref_target_logits, valid_len, row_logp, ref_logp, stream=None) -> None:
    lib = load_library()
    lt = LOGIT_DTYPES[params.dtype]
    st = lib.ppow_reference_logprob(ctypes.byref(params), _dev_ptr(ref_target_logits, lt, "ref_target_logits"),
                                    _dev_ptr(valid_len, torch.int32, "valid_len"),
                                    _dev_ptr(row_logp, torch.float32, "row_logp"),
                                    _dev_ptr(ref_logp, torch.float32, "ref_logp"), _stream_ptr(stream))
    if st != PPOW_OK:
        raise PpowError(st, "ppow_reference_logprob")


def _host_ptr(t: Optional[torch.Tensor], dtype=None, name="tensor"):
    if t is None:
        return None
    if t.is_cuda or not t.is_contiguous():
        raise ValueError("%s must be a contiguous host tensor" % name)
    if dtype is not None and t.dtype != dtype:
        raise ValueError("%s must have dtype %s, got %s" % (name, dtype, t.dtype))
    return ctypes.c_void_p(t.data_ptr())


def ppow_host_scratch_bytes(params: ppow_params, chunk_windows: int) -> int:
    return int(load_library().ppow_host_scratch_bytes(ctypes.byref(params), int(chunk_windows)))


def ppow_score_and_select_host(params: ppow_params, draft_logits, target_logits, draft_tokens, uniforms, valid_len,
                               ref_logp, outputs_host: dict, n_keep: int, selected_host, mask_host,
                               device_scratch: torch.Tensor, stream=None) -> None:
    """Host-buffer entry point: all tensors except ``device_scratch`` are host tensors (pinned for async copies)."""
    lib = load_library()
    lt = LOGIT_DTYPES[params.dtype]
    o = ppow_outputs()
    for name, _ in ppow_outputs._fields_:
        want = _ALL_OUTPUTS[name]
        p = _host_ptr(outputs_host.get(name), want, name)
        setattr(o, name, p.value if p is not None else None)
    st = lib.ppow_score_and_select_host(
        ctypes.byref(params), _host_ptr(draft_logits, lt, "draft_logits"), _host_ptr(target_logits, lt, "target_logits"),
        _host_ptr(draft_tokens, torch.int32, "draft_tokens"), _host_ptr(uniforms, torch.float32, "uniforms"),
        _host_ptr(valid_len, torch.int32, "valid_len"), _host_ptr(ref_logp, torch.float32, "ref_logp"),
        ctypes.byref(o), int(n_keep), _host_ptr(selected_host, torch.int32, "selected_host"),
        _host_ptr(mask_host, torch.uint8, "mask_host"), _dev_ptr(device_scratch, torch.uint8, "device_scratch"),
        device_scratch.numel(), _stream_ptr(stream))
    if st != PPOW_OK:
        raise PpowError(st, "ppow_score_and_select_host")


# ---- convenience wrappers (allocation + the calls above; no arithmetic) -----------------------


def score_windows(draft_logits, target_logits, draft_tokens, *, mode, c, temperature=1.0, eta=1.0, eps=0.5,
                  uniforms=None, valid_len=None, ref_logp=None, stream=None, train_outputs=False) -> dict:
    """Allocate outputs and workspace, run ppow_score_windows, return the dict of output tensors
    (with ``train_outputs`` also kl_rev, kl_rev_mean, nabla, lse_p, lse_q)."""
    N, K, V = draft_logits.shape
    dt = DTYPE_CODES[draft_logits.dtype]
    params = make_params(N, K, V, dt, mode, c, temperature, eta, eps)
    dev = draft_logits.device
    with torch.cuda.device(dev):
        out = alloc_outputs(N, K, dev)
        if train_outputs:
            out.update(alloc_train_outputs(N, K, dev))
        ws = alloc_workspace(ppow_score_workspace_bytes(params), dev)
        ppow_score_windows(params, draft_logits, target_logits, draft_tokens, uniforms, valid_len, ref_logp, out,
                           ws, stream)
    out["_workspace"] = ws
    return out


def select_windows(score, n_keep: int, want_mask: bool = False, stream=None):
    """Allocate and run ppow_select_windows; returns selected indices (and the mask if asked)."""
    N = int(score.numel())
    dev = score.device
    with torch.cuda.device(dev):
        sel = torch.empty((max(int(n_keep), 0),), dtype=torch.int32, device=dev)
        mask = torch.empty((N,), dtype=torch.uint8, device=dev) if want_mask else None
        ws = alloc_workspace(ppow_select_workspace_bytes(N), dev)
        ppow_select_windows(score, n_keep, sel, mask, ws, stream)
    return (sel, mask) if want_mask else sel
