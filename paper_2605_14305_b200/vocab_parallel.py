"""Vocabulary-parallel verification: argument marshalling around the four ``fef_vp_*`` calls
(see include/fef.h) and the two small all-gathers between them.

Each rank holds, for every position, the logits of one slice of the vocabulary.  The exchange
is ``6 * B * K`` doubles and ``B`` 16-byte records per rank per call; everything else runs in
the library's kernels on the rank's own slice.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import torch

from . import FEF_ERR_INVALID_ARG, FEF_OK, FefError, VerifyResult, _dtype_code, _require_cuda, _stream_ptr, load

STATS_PER_ROW = 6
CANDIDATE_BYTES = 16


def shard_vocab(V: int, ranks: int, multiple: int = 8) -> List[Tuple[int, int]]:
    """(offset, width) of every rank's slice: offsets are multiples of ``multiple`` (the library
    wants 8), widths differ by at most ``multiple``, the last slice takes the remainder."""
    if V < 1 or ranks < 1 or multiple < 1:
        raise ValueError("V, ranks and multiple must be positive")
    blocks = -(-V // multiple)
    if blocks < ranks:
        raise ValueError("more ranks than blocks of %d vocabulary ids" % multiple)
    out, start = [], 0
    for r in range(ranks):
        nb = blocks // ranks + (1 if r < blocks % ranks else 0)
        end = min(V, start + nb * multiple)
        out.append((start, end - start))
        start = end
    return out


class _Rank:
    """Buffers and sizes of one rank's slice."""

    def __init__(self, q: torch.Tensor, p: torch.Tensor, offset: int, V_local: Optional[int], lib=None):
        self.lib = load() if lib is None else lib   # (a stand-in library object is only given by host-side tests)
        if lib is None:
            _require_cuda(q, p)
        if q.dim() != 3 or q.shape != p.shape or q.dtype != p.dtype or not (q.is_contiguous() and p.is_contiguous()):
            raise FefError(FEF_ERR_INVALID_ARG, "fef_vp_local_stats")
        self.q, self.p, self.offset = q, p, int(offset)
        self.B, self.K, self.ld = q.shape
        self.V = self.ld if V_local is None else int(V_local)
        self.code = _dtype_code(q)
        dev = q.device
        self.workspace = torch.empty(max(int(self.lib.fef_spec_verify_workspace_bytes(self.B, self.K, self.V, self.code)),
                                         256), dtype=torch.uint8, device=dev)
        self.stats = torch.empty((self.B * self.K, STATS_PER_ROW), dtype=torch.float64, device=dev)
        self.tasks = torch.empty(int(self.lib.fef_vp_task_bytes(self.B)), dtype=torch.uint8, device=dev)
        self.cand = torch.zeros((self.B, CANDIDATE_BYTES), dtype=torch.uint8, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)


def _sptr(stream) -> int:
    # (a host-side test with a stand-in library and no CUDA device has no stream to name)
    return 0 if stream is None and not torch.cuda.is_available() else _stream_ptr(stream)


def _check(st: int, where: str):
    if st != FEF_OK:
        raise FefError(st, where)


def _local_stats(r: _Rank, tokens, row_len, T, stream):
    _check(r.lib.fef_vp_local_stats(r.q.data_ptr(), r.p.data_ptr(), tokens.data_ptr(),
                                     None if row_len is None else row_len.data_ptr(), r.B, r.K, r.V, r.ld, r.code,
                                     float(T), r.offset, r.stats.data_ptr(), r.workspace.data_ptr(),
                                     r.workspace.numel(), r.status.data_ptr(), _sptr(stream)), "fef_vp_local_stats")


def _accept(r: _Rank, stats_all, ranks, tokens, row_len, V_total, T, seed, step, out: VerifyResult, stream):
    _check(r.lib.fef_vp_accept(stats_all.data_ptr(), ranks, tokens.data_ptr(),
                                None if row_len is None else row_len.data_ptr(), r.B, r.K, int(V_total), r.code, float(T),
                                int(seed) & 0xFFFFFFFFFFFFFFFF, int(step) & 0xFFFFFFFF, out.accept_len.data_ptr(),
                                out.tokens.data_ptr(), out.conf.data_ptr(), r.tasks.data_ptr(),
                                out.device_status.data_ptr(), _sptr(stream)), "fef_vp_accept")


def _local_residual(r: _Rank, T, seed, step, stream):
    _check(r.lib.fef_vp_local_residual(r.q.data_ptr(), r.p.data_ptr(), r.tasks.data_ptr(), r.B, r.K, r.V, r.ld, r.code,
                                        float(T), int(seed) & 0xFFFFFFFFFFFFFFFF, int(step) & 0xFFFFFFFF, r.offset,
                                        r.cand.data_ptr(), r.workspace.data_ptr(), r.workspace.numel(),
                                        _sptr(stream)), "fef_vp_local_residual")


def _finish(r: _Rank, cand_all, ranks, T, out: VerifyResult, stream):
    _check(r.lib.fef_vp_finish(cand_all.data_ptr(), ranks, r.tasks.data_ptr(), r.B, r.K, r.code, float(T),
                                out.tokens.data_ptr(), out.conf.data_ptr(), _sptr(stream)), "fef_vp_finish")


def _new_result(B, K, dev) -> VerifyResult:
    return VerifyResult(torch.empty(B, dtype=torch.int32, device=dev), torch.empty((B, K), dtype=torch.int32, device=dev),
                        torch.empty((B, K), dtype=torch.float32, device=dev), torch.zeros(1, dtype=torch.int32, device=dev))


def fef_spec_verify_vocab_parallel(draft_slice: torch.Tensor, target_slice: torch.Tensor, draft_tokens: torch.Tensor,
                                   temperature: float, seed: int, step: int, vocab_offset: int, V_total: int,
                                   row_len: Optional[torch.Tensor] = None, V_local: Optional[int] = None,
                                   group=None, stream=None, lib=None) -> VerifyResult:
    """One verification call on this rank of a ``torch.distributed`` group whose ranks hold the
    slices of the vocabulary (``draft_slice`` / ``target_slice``: ``[B, K, ld_local]``).  Every
    rank returns the same result.  ``device_status`` holds the acceptance step's status; a
    streaming-side error of this rank is raised into it as well.

    The kernels, the two all-gathers and every allocation of the call run on ``stream`` (made the
    current stream for the duration of the call), so they are ordered against each other whichever
    stream the caller was on.  ``lib``: a stand-in for the loaded library (host-side tests only)."""
    import contextlib

    import torch.distributed as dist

    ranks = dist.get_world_size(group)
    on_stream = torch.cuda.stream(stream) if stream is not None else contextlib.nullcontext()
    with on_stream:
        r = _Rank(draft_slice, target_slice, vocab_offset, V_local, lib)
        out = _new_result(r.B, r.K, draft_slice.device)
        _local_stats(r, draft_tokens, row_len, temperature, stream)
        # (gathered by concatenation along the first axis: rank-major, the layout the next call reads)
        stats_all = torch.empty((ranks * r.stats.shape[0], STATS_PER_ROW), dtype=torch.float64, device=r.stats.device)
        dist.all_gather_into_tensor(stats_all, r.stats, group=group)
        _accept(r, stats_all, ranks, draft_tokens, row_len, V_total, temperature, seed, step, out, stream)
        _local_residual(r, temperature, seed, step, stream)
        cand_all = torch.empty((ranks * r.B, CANDIDATE_BYTES), dtype=torch.uint8, device=r.cand.device)
        dist.all_gather_into_tensor(cand_all, r.cand, group=group)
        _finish(r, cand_all, ranks, temperature, out, stream)
        torch.maximum(out.device_status, r.status, out=out.device_status)
    return out


def fef_spec_verify_sharded_on_one_device(slices: Sequence[Tuple[torch.Tensor, torch.Tensor, int]],
                                          draft_tokens: torch.Tensor, temperature: float, seed: int, step: int,
                                          V_total: int, row_len: Optional[torch.Tensor] = None) -> List[VerifyResult]:
    """The same four steps for all ranks' slices on one GPU, one rank after the other, with the
    gathers done by concatenation: the single-GPU stand-in for the distributed call (kernels of
    different ranks never wait for each other).  ``slices``: (draft_slice, target_slice,
    vocab_offset[, V_local]) per rank; V_local defaults to the slice tensors' row pitch.  Returns every rank's result (they must be identical)."""
    ranks = [_Rank(t[0], t[1], t[2], t[3] if len(t) > 3 else None) for t in slices]
    n = len(ranks)
    dev = draft_tokens.device
    for r in ranks:
        _local_stats(r, draft_tokens, row_len, temperature, None)
    stats_all = torch.stack([r.stats for r in ranks]).contiguous()
    outs = [_new_result(ranks[0].B, ranks[0].K, dev) for _ in ranks]
    for r, out in zip(ranks, outs):
        _accept(r, stats_all, n, draft_tokens, row_len, V_total, temperature, seed, step, out, None)
        _local_residual(r, temperature, seed, step, None)
    cand_all = torch.stack([r.cand for r in ranks]).contiguous()
    for r, out in zip(ranks, outs):
        _finish(r, cand_all, n, temperature, out, None)
        torch.maximum(out.device_status, r.status, out=out.device_status)
    return outs
