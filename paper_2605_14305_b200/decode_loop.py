"""Host-side driver of the paper's full-sequence decoding loop (Algorithm 2) around
the two library calls, for tests and benchmarks.

The models are replaced by a caller-supplied ``logits_fn`` that returns the draft
and target logits of the current speculative windows; everything the paper's loop
does besides the two library calls is bookkeeping on small integer arrays, kept
on the host here:

  for s = 0 .. n_steps-1:                       (denoising steps)
      C <- {}                                   (positions committed during this step)
      while some position is unresolved:        (speculative rounds)
          window = first min(K, #unresolved) unresolved positions of each batch row
          verify(window)  -> commit accepted drafts and the corrected token, record c_j
      if s < n_steps-1: R = LowConf_k(C); re-mask the positions in R

Re-corruption uses the absorbing-state forward kernel: a selected position goes
back to [MASK] (stored as -1).  ``verify_fn`` and ``select_fn`` are injected so the
same driver can run any implementation.
"""
from __future__ import annotations

import time
from typing import Callable, Optional

import numpy as np
import torch

MASK = -1


def run_decode_loop(B: int, L: int, K: int, n_steps: int, remask_k: int,
                    logits_fn: Callable, draft_fn: Callable, verify_fn: Callable, select_fn: Callable,
                    on_round: Optional[Callable] = None, device="cuda", first_round: int = 0):
    """Run Algorithm 2 on ``B`` sequences of ``L`` positions that all start masked.

    logits_fn(round, window_pos [B,K] int64 (-1 = unused), row_len [B]) -> (draft_logits, target_logits)  [B,K,V]
    draft_fn(draft_logits, round) -> draft_tokens [B,K] int32
    verify_fn(draft_logits, target_logits, draft_tokens, row_len int32 [B] tensor, round)
        -> (accept_len [B], tokens [B,K], conf [B,K]) as host numpy arrays
    select_fn(conf [B,L] float32 tensor, mask [B,L] uint8 tensor, k) -> (positions [B,k], count [B]) numpy
    on_round(round, inputs, outputs): optional hook (parity checks)

    Returns dict(tokens [B,L], conf [B,L], rounds, committed_per_round list).
    """
    tokens = np.full((B, L), MASK, dtype=np.int64)
    conf = np.full((B, L), -1.0, dtype=np.float32)
    rnd = first_round
    committed_hist = []
    for s in range(n_steps):
        in_C = np.zeros((B, L), dtype=np.uint8)
        while (tokens == MASK).any():
            window = np.full((B, K), -1, dtype=np.int64)
            row_len = np.zeros(B, dtype=np.int32)
            for b in range(B):
                unresolved = np.nonzero(tokens[b] == MASK)[0][:K]
                row_len[b] = len(unresolved)
                window[b, :len(unresolved)] = unresolved
            q, p = logits_fn(rnd, window, row_len)
            draft = draft_fn(q, rnd)
            rl = torch.as_tensor(row_len, device=device)
            accept_len, out_tok, out_conf = verify_fn(q, p, draft, rl, rnd)
            if on_round is not None:
                on_round(rnd, (q, p, draft, rl), (accept_len, out_tok, out_conf))
            n_committed = 0
            for b in range(B):
                if accept_len[b] < 0:
                    raise RuntimeError("verification reported a data error in window %d" % b)
                m = min(int(accept_len[b]) + 1, int(row_len[b]))
                pos = window[b, :m]
                tokens[b, pos] = out_tok[b, :m]
                conf[b, pos] = out_conf[b, :m]
                in_C[b, pos] = 1
                n_committed += m
            committed_hist.append(n_committed)
            rnd += 1
        if s < n_steps - 1 and remask_k > 0:
            positions, count = select_fn(torch.as_tensor(conf, device=device), torch.as_tensor(in_C, device=device),
                                         remask_k)
            for b in range(B):
                sel = positions[b, :count[b]]
                tokens[b, sel] = MASK
                conf[b, sel] = -1.0
    return dict(tokens=tokens, conf=conf, rounds=rnd - first_round, committed_per_round=committed_hist)


def run_decode_loop_device(fef, B: int, L: int, K: int, n_steps: int, remask_k: int, logits_fn: Callable,
                           temperature: float, seed: int, on_round: Optional[Callable] = None,
                           first_round: int = 0, reuse_draft_norm: bool = True, build_inputs: bool = False,
                           reuse_target_norm: bool = False, V: Optional[int] = None):
    """Algorithm 2 with the whole state resident on the device: every step of a round is one
    library call (``fef_loop_next_window`` -> [``fef_loop_verification_inputs``] ->
    ``fef_draft_sample`` -> ``fef_spec_verify`` -> ``fef_loop_commit``), and a denoising step ends
    with ``fef_remask_select`` + ``fef_loop_remask``.  The host reads back one integer per round
    (the largest count of unresolved positions) to know when the step is over.

    ``fef`` is the binding module.  logits_fn(round, window_pos [B,K] int32 CUDA, row_len [B] int32
    CUDA, inputs [B,K,L] int32 CUDA or None) -> (draft_logits, target_logits), both [B,K,V] CUDA.
    on_round(round, dict of the round's device tensors): optional hook, called after the commit with
    the state before it under "before"; called with round None after each re-masking.
    reuse_target_norm: the draft draws also reduce the target rows (``fef_draft_sample(target_logits=)``)
    and the verification takes both normalisers, so both tensors are read once per round.
    V: vocabulary size when the logits' row pitch is larger.

    Returns dict(tokens [B,L] int32, conf [B,L] float32 (CUDA), rounds, committed_per_round, loop_seconds).
    """
    dev = torch.device("cuda")
    tokens = torch.full((B, L), MASK, dtype=torch.int32, device=dev)
    conf = torch.full((B, L), -1.0, dtype=torch.float32, device=dev)
    in_step = torch.zeros((B, L), dtype=torch.uint8, device=dev)
    rnd = first_round
    committed_hist = []
    torch.cuda.synchronize()
    t_start = time.perf_counter()
    for s in range(n_steps):
        while True:
            window, row_len, unresolved = fef.fef_loop_next_window(tokens, K)
            if int(unresolved.max().item()) == 0:
                break
            inputs = None
            q, p = logits_fn(rnd, window, row_len, None)
            draft = fef.fef_draft_sample(q, temperature, seed, rnd, row_len=row_len, V=V,
                                         target_logits=p if reuse_target_norm else None)
            if build_inputs:
                inputs = fef.fef_loop_verification_inputs(tokens, window, row_len, draft.tokens)
            norm = draft.log2_norm if (reuse_draft_norm or reuse_target_norm) else None
            res = fef.fef_spec_verify(q, p, draft.tokens, temperature, seed, rnd, row_len=row_len, V=V,
                                      draft_log2_norm=norm,
                                      target_log2_norm=draft.target_log2_norm if reuse_target_norm else None)
            before = (tokens.clone(), conf.clone(), in_step.clone()) if on_round is not None else None
            committed = fef.fef_loop_commit(window, row_len, res, tokens, conf, in_step)
            if on_round is not None:
                on_round(rnd, dict(q=q, p=p, draft=draft, window=window, row_len=row_len, unresolved=unresolved,
                                   inputs=inputs, result=res, committed=committed, before=before,
                                   tokens=tokens, conf=conf, in_step=in_step))
            n = committed.cpu()
            if (n < 0).any():
                raise RuntimeError("verification reported a data error in round %d" % rnd)
            committed_hist.append(int(n.sum()))
            rnd += 1
        if s < n_steps - 1 and remask_k > 0:
            positions, count = fef.fef_remask_select(conf, in_step, remask_k)
            before = (tokens.clone(), conf.clone(), in_step.clone()) if on_round is not None else None
            fef.fef_loop_remask(positions, count, tokens, conf, in_step)
            if on_round is not None:
                on_round(None, dict(positions=positions, count=count, before=before,
                                    tokens=tokens, conf=conf, in_step=in_step))
    torch.cuda.synchronize()
    return dict(tokens=tokens, conf=conf, rounds=rnd - first_round, committed_per_round=committed_hist,
                loop_seconds=time.perf_counter() - t_start)


def run_decode_loop_graph(fef, B: int, L: int, K: int, n_steps: int, remask_k: int, logits_fn: Callable,
                          temperature: float, seed: int, first_round: int = 0, reuse_draft_norm: bool = True,
                          rounds_per_check: int = 4):
    """``run_decode_loop_device`` with one whole round captured as a CUDA graph and replayed.

    The round's number lives in a device word that ``fef_draft_sample`` / ``fef_spec_verify`` add
    to their step (``device_round=``) and ``fef_loop_advance_round`` bumps while some row still
    has unresolved positions, so every replay draws the random numbers the eager loop would.  The
    host launches ``rounds_per_check`` replays at a time and then reads one integer; replays after
    the last real round of a denoising step change nothing.

    logits_fn(device_round [1] int32 CUDA, window_pos, row_len) -> (draft_logits, target_logits):
    must be capturable (device work only, the round read from the tensor).

    Returns dict(tokens, conf (CUDA), rounds, loop_seconds: wall time of the replay loop alone).
    """
    dev = torch.device("cuda")
    tokens = torch.full((B, L), MASK, dtype=torch.int32, device=dev)
    conf = torch.full((B, L), -1.0, dtype=torch.float32, device=dev)
    in_step = torch.zeros((B, L), dtype=torch.uint8, device=dev)
    rnd = torch.zeros(1, dtype=torch.int32, device=dev)

    def one_round():
        window, row_len, unresolved = fef.fef_loop_next_window(tokens, K)
        q, p = logits_fn(rnd, window, row_len)
        draft = fef.fef_draft_sample(q, temperature, seed, first_round, row_len=row_len, device_round=rnd)
        res = fef.fef_spec_verify(q, p, draft.tokens, temperature, seed, first_round, row_len=row_len,
                                  draft_log2_norm=draft.log2_norm if reuse_draft_norm else None, device_round=rnd)
        fef.fef_loop_commit(window, row_len, res, tokens, conf, in_step)
        fef.fef_loop_advance_round(rnd, unresolved)
        return unresolved

    # one eager round on a side stream first (per-device set-up of the library, allocator warm-up),
    # then the state is put back and the same round is captured
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        one_round()
    torch.cuda.current_stream().wait_stream(side)
    tokens.fill_(MASK)
    conf.fill_(-1.0)
    in_step.zero_()
    rnd.zero_()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        unresolved = one_round()

    torch.cuda.synchronize()
    t_start = time.perf_counter()
    for s in range(n_steps):
        while True:
            for _ in range(rounds_per_check):
                graph.replay()
            if int(unresolved.max().item()) == 0:   # counted before the last replay: nothing was left
                break
        if s < n_steps - 1 and remask_k > 0:
            positions, count = fef.fef_remask_select(conf, in_step, remask_k)
            fef.fef_loop_remask(positions, count, tokens, conf, in_step)
    torch.cuda.synchronize()
    return dict(tokens=tokens, conf=conf, rounds=int(rnd.item()), loop_seconds=time.perf_counter() - t_start)
