"""CPU oracle for the bookkeeping of the paper's full-sequence decoding loop (Algorithm 2).

TEST INFRASTRUCTURE ONLY.  Plain numpy and Python loops, written from Algorithm 2: the ordered
set of unresolved positions J_t and the window size b = min{k, L_t}; the verification inputs
X^(j_m) ("each input uses the verified prefix and the draft prefix x~_{j_1..j_{m-1}}"); the
write-back of accepted and corrected tokens with their confidences into X and C^(s); and the
re-corruption of the positions LowConf selected (absorbing-state kernel: back to [MASK]).
Shares no code with the CUDA library.  MASK is token id -1.

Pins (tests/test_oracle_pins.py): window positions against numpy's nonzero; the inputs against the
definition spelled out per position on small cases; the committed count against Theorem 2's
"accepted drafts plus the corrected position"; a full toy loop terminates with every position
resolved and the re-masked set equal to a library sort's k smallest.
"""
from __future__ import annotations

import numpy as np

MASK = -1


def next_window(tokens, K):
    """tokens [B, L] -> (window_pos [B, K] int32, -1 = unused; row_len [B]; unresolved [B])."""
    tokens = np.asarray(tokens)
    B, L = tokens.shape
    window = np.full((B, K), -1, dtype=np.int32)
    row_len = np.zeros(B, dtype=np.int32)
    unresolved = np.zeros(B, dtype=np.int32)
    for b in range(B):
        n = 0
        for j in range(L):                      # J_t in increasing order
            if tokens[b, j] == MASK:
                if n < K:
                    window[b, n] = j
                n += 1
        unresolved[b] = n
        row_len[b] = min(K, n)                  # b = min{k, L_t}
    return window, row_len, unresolved


def verification_inputs(tokens, window_pos, row_len, draft_tokens):
    """X^(j_m) for m = 0 .. K-1: the current sequence with the drafts of the window's earlier
    positions j_0 .. j_{m-1} written in; [B, K, L] int32.  Rows m >= row_len[b] repeat the
    sequence with all of the window's drafts written in (they are not used)."""
    tokens = np.asarray(tokens)
    B, L = tokens.shape
    K = window_pos.shape[1]
    out = np.zeros((B, K, L), dtype=np.int32)
    for b in range(B):
        for m in range(K):
            x = tokens[b].astype(np.int32).copy()
            for mm in range(min(m, int(row_len[b]))):
                x[window_pos[b, mm]] = draft_tokens[b, mm]
            out[b, m] = x
    return out


def commit(tokens, conf, in_step, window_pos, row_len, accept_len, out_tokens, out_conf):
    """Write back one verification call (in place).  Returns committed [B]: accepted drafts plus
    the corrected position, min(a + 1, n); -1 (and nothing written) for a window with a data error."""
    B = tokens.shape[0]
    committed = np.zeros(B, dtype=np.int32)
    for b in range(B):
        a, n = int(accept_len[b]), int(row_len[b])
        if a < 0:
            committed[b] = -1
            continue
        m = min(a + 1, n)
        for t in range(m):
            j = window_pos[b, t]
            tokens[b, j] = out_tokens[b, t]
            conf[b, j] = out_conf[b, t]
            in_step[b, j] = 1                   # C^(s) <- C^(s) u {(j, c_j)}
        committed[b] = m
    return committed


def remask(tokens, conf, in_step, positions, count):
    """Re-corrupt the selected positions (back to MASK) and start the next step's C^(s) empty."""
    B = tokens.shape[0]
    for b in range(B):
        for t in range(int(count[b])):
            j = positions[b, t]
            tokens[b, j] = MASK
            conf[b, j] = -1.0
    in_step[...] = 0
