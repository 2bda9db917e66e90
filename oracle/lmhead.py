"""CPU oracle for verification straight from hidden states (test infrastructure, not the product).

The draft and target laws of Section 3.2 are model outputs: logits = hidden state x output-layer
weight, one row per window position.  Here that product is written out in double precision on the
same bfloat16 bytes the CUDA path reads (a library matrix product is the step; no blocking, no
reduced precision), and the resulting float64 logits go through the verification oracle unchanged
(Algorithm 2's loop over the window's positions).  Shares no code with the CUDA library.

Pins (tests/test_oracle_pins.py): the product against exact integer arithmetic on small
integer-valued inputs and against the identity weight; float64 logit storage against the float32
path on values both can hold exactly.
"""
from __future__ import annotations

import numpy as np

from . import spec_verify


def _as_float64(x) -> np.ndarray:
    """bfloat16 / float32 torch tensor, or a numpy array, as float64 (exact: every input value is representable)."""
    try:
        import torch

        if isinstance(x, torch.Tensor):
            return x.detach().cpu().to(torch.float64).numpy()
    except ImportError:  # pragma: no cover
        pass
    return np.asarray(x, dtype=np.float64)


def lmhead_logits(hidden, weight) -> np.ndarray:
    """logits[r, v] = sum_k hidden[r, k] * weight[v, k] in double precision; hidden [R, d], weight [V, d]."""
    H, W = _as_float64(hidden), _as_float64(weight)
    assert H.ndim == 2 and W.ndim == 2 and H.shape[1] == W.shape[1]
    return H @ W.T


def lmhead_spec_verify(draft_hidden, target_hidden, weight, draft_tokens, B, K, temperature, seed, step, row_len=None,
                       batch_offset=0):
    """The verification oracle on the double-precision logits of the two hidden-state matrices
    (each [B*K, d], row b*K+i = position i of window b).  Returns ``oracle.spec_verify``'s dict plus
    the logits themselves under "draft_logits" / "target_logits" ([B, K, V] float64)."""
    lq = lmhead_logits(draft_hidden, weight)
    lp = lmhead_logits(target_hidden, weight)
    V = lq.shape[1]
    assert lq.shape[0] == B * K and lp.shape == lq.shape
    lq, lp = lq.reshape(B, K, V), lp.reshape(B, K, V)
    out = spec_verify(lq, lp, draft_tokens, temperature, seed, step, row_len=row_len, batch_offset=batch_offset)
    out["draft_logits"], out["target_logits"] = lq, lp
    return out
