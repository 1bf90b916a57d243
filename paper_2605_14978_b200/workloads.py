"""Seeded synthetic inputs for the PPOW window-scoring pass.

This module only makes inputs: paired draft/target logits ``[N, K, V]``, drafted tokens, uniforms
and ragged lengths.  It holds none of the scoring arithmetic and is the one module that both the
CUDA tests/benchmark and the CPU oracle's tests draw their data from.

The logits stand in for what a drafter/target pair emits on dialogue, code and maths prompts (the
paper trains on such data with LLaMA-3 and Qwen3 vocabularies); no dataset or checkpoint is read.

Recipe (all arithmetic in float32, each tensor rounded once to its storage type):
    target[n,k,v] = -ln(rank_{n,k}(v)) + noise          rank_{n,k}: independent uniform permutation of 1..V
    draft         = target_f32 + sigma_k * noise'        sigma_k = lo + (hi-lo) * k/(K-1)
    tokens        ~ Categorical(softmax(draft_stored / T))
    uniforms      ~ U[0,1) float32
Windows are generated in chunks of ``CHUNK`` windows; chunk j of stream s of workload w uses the
seed ``(1000*w + s) * 4096 + j`` so any chunk can be regenerated alone.  Streams: 0 tokens,
1 target, 2 draft noise, 3 uniforms, 4 lengths, 5 hard positions.
"""
from __future__ import annotations

import dataclasses
from typing import Optional, Tuple

import torch

CHUNK = 64  # windows per independently seeded chunk


@dataclasses.dataclass(frozen=True)
class Workload:
    index: int
    name: str
    N: int
    K: int
    V: int
    dtype: str                      # "f32" | "bf16" | "f16"
    noise: str                      # "normal" | "student_t3"
    sigma_lo: float
    sigma_hi: float
    modes: Tuple[str, ...]          # each "greedy" | "stochastic"
    temperature: float
    c: float
    keep_pct: int
    ragged: Optional[Tuple[int, int]] = None   # valid lengths uniform in [lo, hi]
    hard_frac: float = 0.0          # fraction of windows with one forced draft/target argmax mismatch

    @property
    def n_keep(self) -> int:
        return (self.keep_pct * self.N + 99) // 100

    @property
    def torch_dtype(self):
        return {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[self.dtype]

    @property
    def logit_bytes_per_window(self) -> int:
        return 2 * self.K * self.V * (4 if self.dtype == "f32" else 2)


WORKLOADS = (
    Workload(0, "tiny", 64, 4, 1000, "f32", "normal", 0.5, 0.5, ("greedy",), 1.0, 0.05, 25),
    Workload(1, "vicuna_like", 1024, 8, 32000, "bf16", "normal", 0.2, 1.5, ("greedy",), 1.0, 0.05, 25),
    Workload(2, "llama3_like", 2048, 8, 128256, "bf16", "normal", 0.3, 2.0, ("stochastic",), 1.0, 0.04, 25),
    Workload(3, "qwen_like", 4096, 10, 151936, "bf16", "normal", 0.3, 2.0, ("stochastic",), 0.7, 0.05, 10,
             ragged=(4, 10), hard_frac=0.2),
    Workload(4, "heavy_tail", 8192, 12, 152064, "bf16", "student_t3", 0.5, 2.5, ("greedy", "stochastic"),
             1.0, 0.03, 20),
)
BY_NAME = {w.name: w for w in WORKLOADS}


def scaled(w: Workload, N: int, name: Optional[str] = None) -> Workload:
    """The same recipe with a different number of windows (parity samples, CPU-sized cases)."""
    return dataclasses.replace(w, N=N, name=name or ("%s_n%d" % (w.name, N)))


def _gen(w: Workload, stream: int, chunk: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((1000 * w.index + stream) * 4096 + chunk)
    return g


def _noise(w: Workload, shape, g, device) -> torch.Tensor:
    z = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    if w.noise == "normal":
        return z
    # Student-t with 3 degrees of freedom: z / sqrt(chi2_3 / 3)
    chi2 = torch.zeros(shape, device=device, dtype=torch.float32)
    for _ in range(3):
        e = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
        chi2.addcmul_(e, e)
    return z.div_(chi2.div_(3.0).sqrt_())


def generate_chunk(w: Workload, chunk: int, device="cpu") -> dict:
    """Windows [chunk*CHUNK, min(N, (chunk+1)*CHUNK)) of workload ``w`` on ``device``."""
    device = torch.device(device)
    n0 = chunk * CHUNK
    nw = min(w.N, n0 + CHUNK) - n0
    assert nw > 0
    K, V = w.K, w.V
    shape = (nw, K, V)

    g_t = _gen(w, 1, chunk, device)
    keys = torch.rand(shape, generator=g_t, device=device, dtype=torch.float32)
    rank = keys.argsort(dim=-1).add_(1).to(torch.float32)
    del keys
    target32 = rank.log_().neg_()
    target32.add_(_noise(w, shape, g_t, device))

    g_d = _gen(w, 2, chunk, device)
    if K > 1:
        sigma = w.sigma_lo + (w.sigma_hi - w.sigma_lo) * torch.arange(K, device=device, dtype=torch.float32) / (K - 1)
    else:
        sigma = torch.full((1,), w.sigma_lo, device=device, dtype=torch.float32)
    draft32 = _noise(w, shape, g_d, device).mul_(sigma.view(1, K, 1)).add_(target32)

    valid_len = None
    if w.ragged is not None:
        g_l = _gen(w, 4, chunk, device)
        valid_len = torch.randint(w.ragged[0], w.ragged[1] + 1, (nw,), generator=g_l, device=device,
                                  dtype=torch.int32)

    if w.hard_frac > 0.0:
        g_h = _gen(w, 5, chunk, device)
        is_hard = torch.rand((nw,), generator=g_h, device=device) < w.hard_frac
        L = valid_len.to(torch.int64) if valid_len is not None else torch.full((nw,), K, device=device)
        h = (torch.rand((nw,), generator=g_h, device=device) * L).to(torch.int64).clamp_(max=K - 1)
        h = torch.minimum(h, (L - 1).clamp_(min=0))
        shift = torch.randint(1, V, (nw,), generator=g_h, device=device)
        rows = torch.nonzero(is_hard).flatten()
        if rows.numel() > 0:
            hh = h[rows]
            t_arg = target32[rows, hh].argmax(dim=-1)
            j = (t_arg + shift[rows]) % V                      # any vocab entry except the target argmax
            top = draft32[rows, hh].max(dim=-1).values
            draft32[rows, hh, j] = top + 4.0

    target = target32.to(w.torch_dtype)
    draft = draft32.to(w.torch_dtype)
    del target32, draft32

    g_y = _gen(w, 0, chunk, device)
    probs = torch.softmax(draft.to(torch.float32).view(nw * K, V) / w.temperature, dim=-1)
    tokens = torch.multinomial(probs, 1, generator=g_y).view(nw, K).to(torch.int32)
    del probs

    g_u = _gen(w, 3, chunk, device)
    uniforms = torch.rand((nw, K), generator=g_u, device=device, dtype=torch.float32)
    return {"draft_logits": draft, "target_logits": target, "draft_tokens": tokens, "uniforms": uniforms,
            "valid_len": valid_len}


def generate(w: Workload, device="cpu", chunks=None) -> dict:
    """All windows of ``w`` (or the listed chunks, concatenated in the given order) on ``device``."""
    device = torch.device(device)
    n_chunks = (w.N + CHUNK - 1) // CHUNK
    chunks = list(range(n_chunks)) if chunks is None else list(chunks)
    sizes = [min(w.N, (c + 1) * CHUNK) - c * CHUNK for c in chunks]
    total = sum(sizes)
    out = {
        "draft_logits": torch.empty((total, w.K, w.V), dtype=w.torch_dtype, device=device),
        "target_logits": torch.empty((total, w.K, w.V), dtype=w.torch_dtype, device=device),
        "draft_tokens": torch.empty((total, w.K), dtype=torch.int32, device=device),
        "uniforms": torch.empty((total, w.K), dtype=torch.float32, device=device),
        "valid_len": torch.empty((total,), dtype=torch.int32, device=device) if w.ragged else None,
    }
    pos = 0
    for c, sz in zip(chunks, sizes):
        part = generate_chunk(w, c, device)
        for key, dst in out.items():
            if dst is not None:
                dst[pos:pos + sz].copy_(part[key])
        del part
        pos += sz
    return out
