"""Seeded synthetic inputs for the verification step.

These generators stand in for the logits a draft model (token-wise clean-token
predictor) and a target model (prefix-conditioned predictor) would produce for
a speculative window; no model, dataset or checkpoint is involved.  They are
the ONLY code shared by the CUDA path's tests, the CPU oracle's tests and the
benchmark, and they contain none of the verification step's arithmetic: logits
are drawn, draft tokens are drawn from the draft logits, nothing else.

The same tensors (the same bytes) are handed to both implementations; values
are never regenerated separately on host and device.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional, Tuple

import torch


@dataclass(frozen=True)
class Workload:
    """Shape and value recipe of one verification call."""

    name: str
    B: int
    K: int
    V: int
    dtype: torch.dtype
    family: str          # "gauss" | "peaked" | "zipf"
    draft_std: float     # std of the draft logits
    noise_std: float     # target = draft + N(0, noise_std^2)
    temperature: float
    remask_k: int
    gen_len: int         # generation length of the denoise loop (positions per batch row)

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)

    @property
    def logit_bytes(self) -> int:
        return 2 if self.dtype == torch.bfloat16 else 4


# The five benchmark configurations (vocabulary sizes of LLaDA-8B and Dream-7B).
TINY = Workload("tiny", 1, 4, 1024, torch.float32, "gauss", 1.0, 0.5, 1.0, 2, 4)
LLADA_SINGLE = Workload("llada_single", 1, 32, 126464, torch.bfloat16, "peaked", 2.0, 0.7, 1.0, 8, 256)
LLADA_BATCHED = Workload("llada_batched", 16, 32, 126464, torch.bfloat16, "peaked", 2.0, 0.7, 0.7, 8, 32)
DREAM_LARGE = Workload("dream_large", 64, 32, 152064, torch.bfloat16, "zipf", 2.0, 0.5, 1.0, 8, 32)
HEADLINE = Workload("headline", 64, 32, 126464, torch.bfloat16, "peaked", 2.0, 0.7, 1.0, 8, 1024)

CONFIGS = {w.name: w for w in (TINY, LLADA_SINGLE, LLADA_BATCHED, DREAM_LARGE, HEADLINE)}


def _generator(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def make_logits(w: Workload, seed: int, device="cpu", rows_per_chunk: int = 256) -> Tuple[torch.Tensor, torch.Tensor]:
    """Draft and target logits ``[B, K, V]`` of dtype ``w.dtype`` on ``device``.

    gauss : draft ~ N(0, draft_std^2)
    peaked: draft ~ N(0, draft_std^2), a random 1 % of each row's entries raised by 8
    zipf  : draft ~ N(0, draft_std^2) - 1.1 * ln(1 + v)   (log of a Zipf(1.1) weight on vocabulary id v)
    target = draft + N(0, noise_std^2); both rounded to ``w.dtype`` afterwards.
    Generated in chunks of rows so the fp32 temporaries stay small.
    """
    dev = torch.device(device)
    g = _generator(dev, seed)
    rows = w.B * w.K
    q = torch.empty((rows, w.V), dtype=w.dtype, device=dev)
    p = torch.empty((rows, w.V), dtype=w.dtype, device=dev)
    bias = None
    if w.family == "zipf":
        bias = -1.1 * torch.log1p(torch.arange(w.V, device=dev, dtype=torch.float32))
    for r0 in range(0, rows, rows_per_chunk):
        r1 = min(rows, r0 + rows_per_chunk)
        d = torch.randn((r1 - r0, w.V), generator=g, device=dev, dtype=torch.float32) * w.draft_std
        if w.family == "peaked":
            boost = torch.rand((r1 - r0, w.V), generator=g, device=dev) < 0.01
            d = d + 8.0 * boost.to(torch.float32)
        elif w.family == "zipf":
            d = d + bias
        elif w.family != "gauss":
            raise ValueError("unknown family %r" % w.family)
        t = d + torch.randn((r1 - r0, w.V), generator=g, device=dev, dtype=torch.float32) * w.noise_std
        q[r0:r1] = d.to(w.dtype)
        p[r0:r1] = t.to(w.dtype)
    return q.view(w.B, w.K, w.V), p.view(w.B, w.K, w.V)


def sample_draft_tokens(draft_logits: torch.Tensor, temperature: float, seed: int, rows_per_chunk: int = 256) -> torch.Tensor:
    """Draft tokens ``[B, K]`` (int32), one draw per position from the draft law.

    The draw perturbs ``logits / T`` with Gumbel noise from torch's seeded
    generator and takes the arg-max; at ``T == 0`` it is the plain arg-max.
    """
    B, K, V = draft_logits.shape
    dev = draft_logits.device
    flat = draft_logits.reshape(B * K, V)
    out = torch.empty(B * K, dtype=torch.int64, device=dev)
    g = _generator(dev, seed)
    for r0 in range(0, B * K, rows_per_chunk):
        r1 = min(B * K, r0 + rows_per_chunk)
        x = flat[r0:r1].to(torch.float32)
        if temperature > 0:
            u = torch.rand(x.shape, generator=g, device=dev, dtype=torch.float32)
            u = u.clamp_(1e-12, 1.0 - 1e-7)
            x = x / temperature - torch.log(-torch.log(u))
        out[r0:r1] = torch.argmax(x, dim=-1)
    return out.to(torch.int32).view(B, K)


def make_call(w: Workload, seed: int, device="cpu", noise_std: Optional[float] = None):
    """(draft_logits, target_logits, draft_tokens) for one call of workload ``w``."""
    if noise_std is not None:
        w = w.with_(noise_std=noise_std)
    q, p = make_logits(w, seed, device)
    tok = sample_draft_tokens(q, w.temperature, seed + 7919)
    return q, p, tok


def algorithmic_bytes(w: Workload, rejected_rows: int = 0) -> int:
    """Bytes one verification call has to move: each of the B*K target and draft
    rows once (at T == 0 the draft rows are not needed), the draft token, the
    outputs; plus one more pass over the two rows of every window that rejects."""
    rows = w.B * w.K
    per_row = (2 if w.temperature > 0 else 1) * w.V * w.logit_bytes
    resid = 2 * w.V * w.logit_bytes if w.temperature > 0 else 0
    return rows * (per_row + 4 + 8) + rejected_rows * resid + w.B * 4


def human_bytes(n: float) -> str:
    for unit in ("B", "KB", "MB", "GB"):
        if abs(n) < 1000.0 or unit == "GB":
            return "%.3g %s" % (n, unit)
        n /= 1000.0
    return "%g" % n


__all__ = [
    "Workload", "CONFIGS", "TINY", "LLADA_SINGLE", "LLADA_BATCHED", "DREAM_LARGE", "HEADLINE",
    "make_logits", "sample_draft_tokens", "make_call", "algorithmic_bytes", "human_bytes",
]
