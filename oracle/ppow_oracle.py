"""ctypes front end of the float64 CPU oracle (``ppow_oracle.c``).

Test infrastructure only: imported by ``tests/``, by the smoke check and by the benchmark's
CPU-baseline leg.  Nothing in the product package imports this module, and this module imports
nothing from the product package.

The wrapper only marshals arguments; every number is computed in the C file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ppow_oracle.c")
_LIB = os.path.join(_HERE, "libppow_oracle.so")
_lock = threading.Lock()
_lib = None

F32, BF16, F16 = 0, 1, 2
GREEDY, STOCHASTIC = 0, 1

POSITION_FIELDS = ("accept_flag", "alpha", "entropy", "kl", "conf", "crit", "logp_tok", "logq_tok",
                   "logp_max", "target_argmax")
WINDOW_FIELDS = ("accepted_len", "reward_speedup", "reward_dist", "reward", "delta", "score")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, no fast-math) into a shared object beside its source."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-pthread", "-Wall", "-Wextra",
                   "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True, capture_output=True, text=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        P = ctypes.c_void_p
        lib.ppow_oracle_score.restype = ctypes.c_int
        lib.ppow_oracle_score.argtypes = (
            [ctypes.c_int32] * 5 + [ctypes.c_double] * 4 + [P] * 6 + [P] * 10 + [P] * 6 + [ctypes.c_int32])
        lib.ppow_oracle_select.restype = ctypes.c_int
        lib.ppow_oracle_select.argtypes = [P, ctypes.c_int32, ctypes.c_int32, P, P]
        lib.ppow_oracle_tau_cumprod.restype = ctypes.c_int32
        lib.ppow_oracle_tau_cumprod.argtypes = [P, ctypes.c_int32]
        lib.ppow_oracle_diagnostics.restype = ctypes.c_int
        lib.ppow_oracle_diagnostics.argtypes = [ctypes.c_int32] * 4 + [ctypes.c_double] + [P] * 8 + [ctypes.c_int32]
        lib.ppow_oracle_group_advantage.restype = ctypes.c_int
        lib.ppow_oracle_group_advantage.argtypes = [P, ctypes.c_int32, ctypes.c_int32, ctypes.c_double, P]
        lib.ppow_oracle_sliding_scores.restype = ctypes.c_int32
        lib.ppow_oracle_sliding_scores.argtypes = [P, ctypes.c_int32, ctypes.c_int32, P]
        lib.ppow_oracle_reference_logprob.restype = ctypes.c_int
        lib.ppow_oracle_reference_logprob.argtypes = [ctypes.c_int32] * 4 + [ctypes.c_double] + [P] * 3
        lib.ppow_oracle_decode.restype = ctypes.c_int
        lib.ppow_oracle_decode.argtypes = [P, ctypes.c_int32, ctypes.c_int64, P]
        lib.ppow_oracle_sample_start.restype = ctypes.c_int32
        lib.ppow_oracle_sample_start.argtypes = [P, ctypes.c_int32, ctypes.c_double]
        lib.ppow_oracle_sample_start_mixed.restype = ctypes.c_int32
        lib.ppow_oracle_sample_start_mixed.argtypes = [P, ctypes.c_int32] + [ctypes.c_double] * 3
        _lib = lib
    return _lib


def _as_numpy_logits(x):
    """Accept a numpy float32 / float16 / uint16 (bf16 bits) array or a CPU torch float32 / bfloat16 / float16 tensor."""
    if not isinstance(x, np.ndarray):
        import torch
        assert isinstance(x, torch.Tensor) and x.device.type == "cpu"
        x = x.contiguous()
        if x.dtype == torch.bfloat16:
            x = x.view(torch.int16).numpy().view(np.uint16)
        elif x.dtype in (torch.float32, torch.float16):
            x = x.numpy()
        else:
            raise TypeError("logits must be float32, bfloat16 or float16")
    x = np.ascontiguousarray(x)
    if x.dtype == np.float32:
        return x, F32
    if x.dtype == np.uint16:
        return x, BF16
    if x.dtype == np.float16:
        return x.view(np.uint16), F16
    raise TypeError("logits must be float32, float16 or uint16 (bf16 bit patterns)")


def _np(x, dtype):
    if x is None:
        return None
    if not isinstance(x, np.ndarray):
        x = x.detach().cpu().numpy()
    return np.ascontiguousarray(x, dtype=dtype)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def score_windows(draft_logits, target_logits, draft_tokens, *, mode, c, temperature=1.0, eta=1.0,
                  eps=0.5, uniforms=None, valid_len=None, ref_logp=None, n_threads=None):
    """Score N windows of K positions over a vocabulary of V entries; returns a dict of numpy arrays.

    Per-position arrays are [N, K]; per-window arrays are [N].  All floating-point results are
    float64.  ``uniforms`` are float32 values supplied by the caller (App. C.1 draws u_t ~ U(0,1));
    the oracle draws no random numbers itself.
    """
    lib = _load()
    d, dt_d = _as_numpy_logits(draft_logits)
    t, dt_t = _as_numpy_logits(target_logits)
    assert dt_d == dt_t and d.shape == t.shape and d.ndim == 3
    N, K, V = d.shape
    tok = _np(draft_tokens, np.int32)
    assert tok.shape == (N, K)
    u = _np(uniforms, np.float32)
    vl = _np(valid_len, np.int32)
    rl = _np(ref_logp, np.float64)
    if n_threads is None:
        n_threads = os.cpu_count() or 1
    out = {
        "accept_flag": np.zeros((N, K), np.uint8),
        "target_argmax": np.zeros((N, K), np.int32),
        "accepted_len": np.zeros((N,), np.int32),
    }
    for f in POSITION_FIELDS:
        out.setdefault(f, np.zeros((N, K), np.float64))
    for f in WINDOW_FIELDS:
        out.setdefault(f, np.zeros((N,), np.float64))
    rc = lib.ppow_oracle_score(
        N, K, V, dt_d, int(mode), float(c), float(temperature), float(eta), float(eps),
        _ptr(d), _ptr(t), _ptr(tok), _ptr(u), _ptr(vl), _ptr(rl),
        *[_ptr(out[f]) for f in POSITION_FIELDS],
        *[_ptr(out[f]) for f in WINDOW_FIELDS],
        int(n_threads))
    if rc != 0:
        raise RuntimeError("ppow_oracle_score failed with code %d" % rc)
    return out


def select_windows(score, n_keep, want_mask=False):
    """Indices of the n_keep largest scores, ordered by (score descending, index ascending)."""
    lib = _load()
    s = _np(score, np.float64)
    N = s.shape[0]
    sel = np.zeros((max(n_keep, 0),), np.int32)
    mask = np.zeros((N,), np.uint8) if want_mask else None
    rc = lib.ppow_oracle_select(_ptr(s), N, int(n_keep), _ptr(sel), _ptr(mask))
    if rc != 0:
        raise RuntimeError("ppow_oracle_select failed with code %d" % rc)
    return (sel, mask) if want_mask else sel


def tau_cumprod(flags):
    """Accepted length by the sum-of-cumulative-products formula of App. C.1."""
    lib = _load()
    f = _np(flags, np.uint8)
    return int(lib.ppow_oracle_tau_cumprod(_ptr(f), int(f.shape[0])))


def diagnostics(draft_logits, target_logits, draft_tokens, *, temperature=1.0, valid_len=None, n_threads=None):
    """Per position: KL(Q||P) (``kl_rev``), expected acceptance sum_v min(P,Q) (``expected_accept``) and the
    alignment divergence exp(d)-d-1 on the drafted token (``nabla``); per window the mean of kl_rev over the
    valid positions (``kl_rev_mean``).  All float64."""
    lib = _load()
    d, dt_d = _as_numpy_logits(draft_logits)
    t, dt_t = _as_numpy_logits(target_logits)
    assert dt_d == dt_t and d.shape == t.shape and d.ndim == 3
    N, K, V = d.shape
    tok = _np(draft_tokens, np.int32)
    vl = _np(valid_len, np.int32)
    out = {"kl_rev": np.zeros((N, K)), "kl_rev_mean": np.zeros((N,)), "nabla": np.zeros((N, K)),
           "expected_accept": np.zeros((N, K))}
    rc = lib.ppow_oracle_diagnostics(N, K, V, dt_d, float(temperature), _ptr(d), _ptr(t), _ptr(tok), _ptr(vl),
                                     _ptr(out["kl_rev"]), _ptr(out["kl_rev_mean"]), _ptr(out["nabla"]),
                                     _ptr(out["expected_accept"]), int(n_threads or os.cpu_count() or 1))
    if rc != 0:
        raise RuntimeError("ppow_oracle_diagnostics failed with code %d" % rc)
    return out


def group_advantage(reward, group_size, delta=1e-6):
    """(R_i - mean) / (population std + delta) within contiguous groups of ``group_size`` windows."""
    lib = _load()
    r = _np(reward, np.float64)
    adv = np.zeros_like(r)
    rc = lib.ppow_oracle_group_advantage(_ptr(r), int(r.shape[0]), int(group_size), float(delta), _ptr(adv))
    if rc != 0:
        raise RuntimeError("ppow_oracle_group_advantage failed with code %d" % rc)
    return adv


def sliding_scores(v, K):
    """s_j = mean(v[j:j+K]) for every start j of one response (empty if it is shorter than K)."""
    lib = _load()
    v = _np(v, np.float64)
    T = int(v.shape[0])
    s = np.zeros((max(T - K + 1, 0),))
    n = lib.ppow_oracle_sliding_scores(_ptr(v), T, int(K), _ptr(s) if s.size else None)
    assert n == s.shape[0]
    return s


def sample_start(s, u):
    """Start index drawn with probability s_j / sum(s) by inverse CDF from the uniform ``u`` (-1: no start)."""
    lib = _load()
    s = _np(s, np.float64)
    return int(lib.ppow_oracle_sample_start(_ptr(s) if s.size else None, int(s.shape[0]), float(u)))


def sample_start_mixed(s, hard_frac, u_mix, u_draw):
    """Hard-window curriculum draw: the ADAW draw ``sample_start(s, u_draw)`` iff ``u_mix < hard_frac``,
    otherwise the uniform start ``floor(u_draw * n)`` (-1: no start)."""
    lib = _load()
    s = _np(s, np.float64)
    return int(lib.ppow_oracle_sample_start_mixed(_ptr(s) if s.size else None, int(s.shape[0]), float(hard_frac),
                                                  float(u_mix), float(u_draw)))


def reference_logprob(ref_logits, *, temperature=1.0, valid_len=None):
    """sum_t max_v log softmax(ref_logits[n,t,:]/T) over the valid positions: the target's log-probability of
    its own greedy reference window (Sec. 4.3.2), given its logits along that window.  float64 [N]."""
    lib = _load()
    r, dt = _as_numpy_logits(ref_logits)
    N, K, V = r.shape
    vl = _np(valid_len, np.int32)
    out = np.zeros((N,))
    rc = lib.ppow_oracle_reference_logprob(N, K, V, dt, float(temperature), _ptr(r), _ptr(vl), _ptr(out))
    if rc != 0:
        raise RuntimeError("ppow_oracle_reference_logprob failed with code %d" % rc)
    return out


def decode(stored):
    """The oracle's own widening of stored logits to float64 (float32 / float16 arrays, uint16 = bf16 bits)."""
    lib = _load()
    a, dt = _as_numpy_logits(stored)
    out = np.zeros(a.shape, np.float64)
    rc = lib.ppow_oracle_decode(_ptr(a), dt, int(a.size), _ptr(out))
    if rc != 0:
        raise RuntimeError("ppow_oracle_decode failed with code %d" % rc)
    return out
