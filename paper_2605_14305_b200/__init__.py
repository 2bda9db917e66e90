"""B200-native speculative verification for FeF-DLLM decoding.

Thin Python binding of the C ABI declared in ``include/fef.h``: the functions
here have the C entry points' names and only marshal arguments (torch tensors
supply device memory and the current stream); every step of the computation
runs in the CUDA library ``libfef.so``.  There is no CPU fallback: calling a
compute function without the built library or without a CUDA device raises.
"""
from __future__ import annotations

import contextlib
import ctypes
import os
from typing import NamedTuple, Optional

import torch

from . import _build

FEF_OK, FEF_ERR_INVALID_ARG, FEF_ERR_DTYPE, FEF_ERR_ALIGNMENT, FEF_ERR_WORKSPACE = 0, 1, 2, 3, 4
FEF_ERR_CUDA, FEF_ERR_TIMEOUT, FEF_ERR_NONFINITE, FEF_ERR_TOKEN_RANGE, FEF_ERR_TOO_LARGE = 5, 6, 7, 8, 9
FEF_STATIC_SCRATCH_BYTES = 8 << 20
FEF_F32, FEF_BF16 = 0, 1
FEF_MAX_K, FEF_MAX_REMASK_L = 64, 8192

EXPORTS = ("fef_status_string", "fef_spec_verify_workspace_bytes", "fef_spec_verify", "fef_spec_verify_profiled",
           "fef_spec_verify_host_arena_bytes", "fef_spec_verify_host", "fef_remask_select",
           "fef_remask_select_host_arena_bytes", "fef_remask_select_host", "fef_spec_verify_static",
           "fef_draft_sample_workspace_bytes", "fef_draft_sample", "fef_spec_verify_with_draft_norm",
           "fef_loop_next_window", "fef_loop_verification_inputs", "fef_loop_commit", "fef_loop_remask",
           "fef_draft_sample_at_round", "fef_spec_verify_at_round", "fef_loop_advance_round",
           "fef_vp_task_bytes", "fef_vp_local_stats", "fef_vp_accept", "fef_vp_local_residual", "fef_vp_finish",
           "fef_lmhead_verify_workspace_bytes", "fef_lmhead_verify", "fef_lmhead_logits",
           "fef_draft_sample_with_target", "fef_spec_verify_with_norms", "fef_synth_logits",
           "fef_loop_run_synthetic_workspace_bytes", "fef_loop_run_synthetic")

_lib = None


class FefError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s (status %d)" % (where, fef_status_string(status), status))


def load(build_if_missing: bool = False) -> ctypes.CDLL:
    """Load ``libfef.so`` (built in-tree by ``_build.build()``).  Raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing:
        _build.build()
    if not os.path.exists(_build.LIB_PATH):
        raise RuntimeError(
            "CUDA library %s is missing: build it with `python -m paper_2605_14305_b200._build` "
            "(there is no CPU fallback)" % _build.LIB_PATH
        )
    L = ctypes.CDLL(_build.LIB_PATH)
    vp, i32, i64, u32, u64, f32, sz = (ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_uint32,
                                       ctypes.c_uint64, ctypes.c_float, ctypes.c_size_t)
    L.fef_status_string.argtypes = [i32]
    L.fef_status_string.restype = ctypes.c_char_p
    L.fef_spec_verify_workspace_bytes.argtypes = [i32, i32, i32, i32]
    L.fef_spec_verify_workspace_bytes.restype = sz
    L.fef_spec_verify.argtypes = [vp, vp, vp, vp, i32, i32, i32, i64, i32, f32, u64, u32, vp, vp, vp, vp, sz, vp, vp]
    L.fef_spec_verify.restype = i32
    L.fef_spec_verify_with_draft_norm.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i64, i32, f32, u64, u32, vp, vp, vp,
                                                  vp, sz, vp, vp]
    L.fef_spec_verify_with_draft_norm.restype = i32
    L.fef_spec_verify_profiled.argtypes = L.fef_spec_verify.argtypes + [vp]
    L.fef_spec_verify_profiled.restype = i32
    L.fef_spec_verify_host_arena_bytes.argtypes = [i32, i32, i32, i64, i32]
    L.fef_spec_verify_host_arena_bytes.restype = sz
    L.fef_spec_verify_host.argtypes = [vp, vp, vp, vp, i32, i32, i32, i64, i32, f32, u64, u32, vp, vp, vp, vp, vp, sz, vp]
    L.fef_spec_verify_host.restype = i32
    L.fef_spec_verify_static.argtypes = [vp, vp, vp, vp, i32, i32, i32, i64, i32, f32, u64, u32, vp, vp, vp, vp, vp]
    L.fef_spec_verify_static.restype = i32
    L.fef_draft_sample_workspace_bytes.argtypes = [i32, i32, i32, i32]
    L.fef_draft_sample_workspace_bytes.restype = sz
    L.fef_draft_sample.argtypes = [vp, vp, i32, i32, i32, i64, i32, f32, u64, u32, vp, vp, vp, sz, vp, vp]
    L.fef_draft_sample.restype = i32
    L.fef_draft_sample_at_round.argtypes = [vp, vp, i32, i32, i32, i64, i32, f32, u64, u32, vp, vp, vp, vp, sz, vp, vp]
    L.fef_draft_sample_at_round.restype = i32
    L.fef_spec_verify_at_round.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i64, i32, f32, u64, u32, vp, vp, vp, vp,
                                           vp, sz, vp, vp]
    L.fef_spec_verify_at_round.restype = i32
    L.fef_draft_sample_with_target.argtypes = [vp, vp, vp, i32, i32, i32, i64, i32, f32, u64, u32, vp, vp, vp, vp, vp, sz,
                                               vp, vp]
    L.fef_draft_sample_with_target.restype = i32
    L.fef_spec_verify_with_norms.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i64, i32, f32, u64, u32, vp, vp, vp, vp,
                                             vp, sz, vp, vp]
    L.fef_spec_verify_with_norms.restype = i32
    L.fef_synth_logits.argtypes = [vp, vp, i32, i32, i32, i64, i32, f32, f32, f32, f32, u64, u32, vp, vp]
    L.fef_synth_logits.restype = i32
    L.fef_loop_run_synthetic_workspace_bytes.argtypes = [i32, i32, i32, i32, i32, i32]
    L.fef_loop_run_synthetic_workspace_bytes.restype = sz
    L.fef_loop_run_synthetic.argtypes = [i32, i32, i32, i32, i32, f32, u64, i32, i32, f32, f32, f32, f32, vp, vp, vp, vp,
                                         vp, sz, vp, vp]
    L.fef_loop_run_synthetic.restype = i32
    L.fef_loop_advance_round.argtypes = [vp, vp, i32, vp]
    L.fef_loop_advance_round.restype = i32
    L.fef_vp_task_bytes.argtypes = [i32]
    L.fef_vp_task_bytes.restype = sz
    L.fef_vp_local_stats.argtypes = [vp, vp, vp, vp, i32, i32, i32, i64, i32, f32, i32, vp, vp, sz, vp, vp]
    L.fef_vp_local_stats.restype = i32
    L.fef_vp_accept.argtypes = [vp, i32, vp, vp, i32, i32, i32, i32, f32, u64, u32, vp, vp, vp, vp, vp, vp]
    L.fef_vp_accept.restype = i32
    L.fef_vp_local_residual.argtypes = [vp, vp, vp, i32, i32, i32, i64, i32, f32, u64, u32, i32, vp, vp, sz, vp]
    L.fef_vp_local_residual.restype = i32
    L.fef_vp_finish.argtypes = [vp, i32, vp, i32, i32, i32, f32, vp, vp, vp]
    L.fef_vp_finish.restype = i32
    L.fef_loop_next_window.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp]
    L.fef_loop_verification_inputs.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp, vp]
    L.fef_loop_commit.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, vp]
    L.fef_loop_remask.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, vp]
    for fn in (L.fef_loop_next_window, L.fef_loop_verification_inputs, L.fef_loop_commit, L.fef_loop_remask):
        fn.restype = i32
    L.fef_lmhead_verify_workspace_bytes.argtypes = [i32, i32, i32, i32]
    L.fef_lmhead_verify_workspace_bytes.restype = sz
    L.fef_lmhead_verify.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, f32, u64, u32, vp, vp, vp, vp, sz, vp, vp]
    L.fef_lmhead_verify.restype = i32
    L.fef_lmhead_logits.argtypes = [vp, vp, i32, i32, i32, vp, i64, vp, vp]
    L.fef_lmhead_logits.restype = i32
    L.fef_remask_select.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp]
    L.fef_remask_select.restype = i32
    L.fef_remask_select_host_arena_bytes.argtypes = [i32, i32, i32]
    L.fef_remask_select_host_arena_bytes.restype = sz
    L.fef_remask_select_host.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, sz, vp]
    L.fef_remask_select_host.restype = i32
    _lib = L
    return L


def fef_status_string(status: int) -> str:
    return load().fef_status_string(int(status)).decode()


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return FEF_F32
    if t.dtype == torch.bfloat16:
        return FEF_BF16
    raise FefError(FEF_ERR_DTYPE, "fef_spec_verify")


def _require_cuda(*tensors):
    if not torch.cuda.is_available():
        raise RuntimeError("no CUDA device: this library has no CPU path")
    for t in tensors:
        if t is not None and t.device.type != "cuda":
            raise ValueError("all tensors must live on a CUDA device")


@contextlib.contextmanager
def _on(device, stream):
    """``device`` current and, when a stream is given, that stream current as well: what a wrapper
    allocates inside (outputs, scratch) then belongs to the stream its kernels run on, so the
    caching allocator cannot hand the memory to someone else while those kernels still use it."""
    with torch.cuda.device(device):
        if stream is None:
            yield
        else:
            with torch.cuda.stream(stream):
                yield


def _stream_ptr(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


def fef_spec_verify_workspace_bytes(B: int, K: int, V: int, dtype) -> int:
    code = dtype if isinstance(dtype, int) else (FEF_F32 if dtype == torch.float32 else FEF_BF16)
    return int(load().fef_spec_verify_workspace_bytes(B, K, V, code))


class VerifyResult(NamedTuple):
    accept_len: torch.Tensor   # [B] int32
    tokens: torch.Tensor       # [B, K] int32
    conf: torch.Tensor         # [B, K] float32
    device_status: torch.Tensor  # [1] int32 (read it after synchronising)


def fef_spec_verify(draft_logits: torch.Tensor, target_logits: torch.Tensor, draft_tokens: torch.Tensor,
                    temperature: float, seed: int, step: int, row_len: Optional[torch.Tensor] = None,
                    V: Optional[int] = None, out: Optional[VerifyResult] = None,
                    workspace: Optional[torch.Tensor] = None, stream=None, stage_events=None,
                    draft_log2_norm: Optional[torch.Tensor] = None,
                    device_round: Optional[torch.Tensor] = None,
                    target_log2_norm: Optional[torch.Tensor] = None) -> VerifyResult:
    """Enqueue one verification call (see ``fef_spec_verify`` in include/fef.h).

    With ``stage_events`` (four ``torch.cuda.Event(enable_timing=True)`` that have
    been recorded once, or ``None`` entries) the call goes through
    ``fef_spec_verify_profiled`` and the events mark the kernel boundaries.  With
    ``draft_log2_norm`` (the ``log2_norm`` of ``fef_draft_sample``, ``[B, K]`` float64) the
    call goes through ``fef_spec_verify_with_draft_norm`` and streams the target rows only.
    With ``target_log2_norm`` as well (from ``fef_draft_sample(..., target_logits=...)``) it goes through
    ``fef_spec_verify_with_norms`` and streams nothing.
    With ``device_round`` (a one-element int32 CUDA tensor) the call goes through
    ``fef_spec_verify_at_round``: the step used is ``step + device_round[0]`` when the kernels run.

    ``draft_logits`` / ``target_logits``: ``[B, K, ld]`` CUDA tensors, float32 or
    bfloat16, contiguous; ``V`` (default ``ld``) entries of each row are used.
    Asynchronous on the current (or given) stream; outputs are reused from
    ``out`` and scratch from ``workspace`` when given.
    """
    _require_cuda(draft_logits, target_logits, draft_tokens, row_len)
    if draft_logits.dim() != 3 or draft_logits.shape != target_logits.shape or draft_logits.dtype != target_logits.dtype:
        raise FefError(FEF_ERR_INVALID_ARG, "fef_spec_verify")
    if not (draft_logits.is_contiguous() and target_logits.is_contiguous() and draft_tokens.is_contiguous()):
        raise FefError(FEF_ERR_INVALID_ARG, "fef_spec_verify")
    if draft_tokens.dtype != torch.int32 or (row_len is not None and row_len.dtype != torch.int32):
        raise FefError(FEF_ERR_INVALID_ARG, "fef_spec_verify")
    B, K, ld = draft_logits.shape
    V = ld if V is None else int(V)
    code = _dtype_code(draft_logits)
    dev = draft_logits.device
    # (nothing to allocate and the device already current: no context to enter, which matters for small calls)
    plain = out is not None and workspace is not None and stream is None and torch.cuda.current_device() == dev.index
    with (contextlib.nullcontext() if plain else _on(dev, stream)):
        if out is None:
            out = VerifyResult(torch.empty(B, dtype=torch.int32, device=dev),
                               torch.empty((B, K), dtype=torch.int32, device=dev),
                               torch.empty((B, K), dtype=torch.float32, device=dev),
                               torch.empty(1, dtype=torch.int32, device=dev))
        if workspace is None:
            workspace = torch.empty(max(fef_spec_verify_workspace_bytes(B, K, V, code), 256),
                                    dtype=torch.uint8, device=dev)
        args = (draft_logits.data_ptr(), target_logits.data_ptr(), draft_tokens.data_ptr(),
                None if row_len is None else row_len.data_ptr(), B, K, V, ld, code, float(temperature),
                int(seed) & 0xFFFFFFFFFFFFFFFF, int(step) & 0xFFFFFFFF,
                out.accept_len.data_ptr(), out.tokens.data_ptr(), out.conf.data_ptr(),
                workspace.data_ptr(), workspace.numel(), out.device_status.data_ptr(), _stream_ptr(stream))
        if draft_log2_norm is not None:
            if draft_log2_norm.dtype != torch.float64 or draft_log2_norm.numel() != B * K or \
                    not draft_log2_norm.is_contiguous() or draft_log2_norm.device != dev:
                raise FefError(FEF_ERR_INVALID_ARG, "fef_spec_verify_with_draft_norm")
        if target_log2_norm is not None:
            if draft_log2_norm is None or target_log2_norm.dtype != torch.float64 or target_log2_norm.numel() != B * K or \
                    not target_log2_norm.is_contiguous() or target_log2_norm.device != dev:
                raise FefError(FEF_ERR_INVALID_ARG, "fef_spec_verify_with_norms")
            if device_round is not None and (device_round.dtype != torch.int32 or device_round.numel() != 1):
                raise FefError(FEF_ERR_INVALID_ARG, "fef_spec_verify_with_norms")
            st = load().fef_spec_verify_with_norms(*args[:3], draft_log2_norm.data_ptr(), target_log2_norm.data_ptr(),
                                                   *args[3:12], None if device_round is None else device_round.data_ptr(),
                                                   *args[12:])
        elif device_round is not None:
            if device_round.dtype != torch.int32 or device_round.numel() != 1 or device_round.device != dev:
                raise FefError(FEF_ERR_INVALID_ARG, "fef_spec_verify_at_round")
            st = load().fef_spec_verify_at_round(*args[:3], None if draft_log2_norm is None else draft_log2_norm.data_ptr(),
                                                 *args[3:12], device_round.data_ptr(), *args[12:])
        elif draft_log2_norm is not None:
            st = load().fef_spec_verify_with_draft_norm(*args[:3], draft_log2_norm.data_ptr(), *args[3:])
        elif stage_events is None:
            st = load().fef_spec_verify(*args)
        else:
            handles = (ctypes.c_void_p * 4)(*[None if e is None else e.cuda_event for e in stage_events])
            st = load().fef_spec_verify_profiled(*args, handles)
    if st != FEF_OK:
        raise FefError(st, "fef_spec_verify")
    return out


class DraftResult(NamedTuple):
    tokens: torch.Tensor         # [B, K] int32, -1 where nothing was drawn
    log2_norm: torch.Tensor      # [B, K] float64
    device_status: torch.Tensor  # [1] int32 (read it after synchronising)
    target_log2_norm: Optional[torch.Tensor] = None  # [B, K] float64, when the target logits were given


def fef_draft_sample_workspace_bytes(B: int, K: int, V: int, dtype) -> int:
    code = dtype if isinstance(dtype, int) else (FEF_F32 if dtype == torch.float32 else FEF_BF16)
    return int(load().fef_draft_sample_workspace_bytes(B, K, V, code))


def fef_draft_sample(draft_logits: torch.Tensor, temperature: float, seed: int, step: int,
                     row_len: Optional[torch.Tensor] = None, V: Optional[int] = None,
                     out: Optional[DraftResult] = None, workspace: Optional[torch.Tensor] = None,
                     stream=None, device_round: Optional[torch.Tensor] = None,
                     target_logits: Optional[torch.Tensor] = None) -> DraftResult:
    """Enqueue the draft-token draws of one call (see ``fef_draft_sample`` in include/fef.h).  With
    ``target_logits`` (same shape and dtype) the call goes through ``fef_draft_sample_with_target`` and
    the result also carries the target laws' normalisers.

    ``draft_logits``: ``[B, K, ld]`` CUDA tensor, float32 or bfloat16, contiguous; ``V`` (default
    ``ld``) entries of each row are used.  Asynchronous on the current (or given) stream.
    """
    _require_cuda(draft_logits, row_len)
    if draft_logits.dim() != 3 or not draft_logits.is_contiguous():
        raise FefError(FEF_ERR_INVALID_ARG, "fef_draft_sample")
    if row_len is not None and row_len.dtype != torch.int32:
        raise FefError(FEF_ERR_INVALID_ARG, "fef_draft_sample")
    B, K, ld = draft_logits.shape
    V = ld if V is None else int(V)
    code = _dtype_code(draft_logits)
    dev = draft_logits.device
    with _on(dev, stream):
        if out is None:
            out = DraftResult(torch.empty((B, K), dtype=torch.int32, device=dev),
                              torch.empty((B, K), dtype=torch.float64, device=dev),
                              torch.empty(1, dtype=torch.int32, device=dev))
        if workspace is None:
            workspace = torch.empty(max(fef_draft_sample_workspace_bytes(B, K, V, code), 256), dtype=torch.uint8,
                                    device=dev)
        head = (draft_logits.data_ptr(), None if row_len is None else row_len.data_ptr(), B, K, V, ld, code,
                float(temperature), int(seed) & 0xFFFFFFFFFFFFFFFF, int(step) & 0xFFFFFFFF)
        tail = (out.tokens.data_ptr(), out.log2_norm.data_ptr(), workspace.data_ptr(), workspace.numel(),
                out.device_status.data_ptr(), _stream_ptr(stream))
        if target_logits is not None:
            _require_cuda(target_logits)
            if target_logits.shape != draft_logits.shape or target_logits.dtype != draft_logits.dtype or \
                    not target_logits.is_contiguous():
                raise FefError(FEF_ERR_INVALID_ARG, "fef_draft_sample_with_target")
            tnorm = out.target_log2_norm
            if tnorm is None:
                tnorm = torch.empty((B, K), dtype=torch.float64, device=dev)
                out = DraftResult(out.tokens, out.log2_norm, out.device_status, tnorm)
            if device_round is not None and (device_round.dtype != torch.int32 or device_round.numel() != 1):
                raise FefError(FEF_ERR_INVALID_ARG, "fef_draft_sample_with_target")
            st = load().fef_draft_sample_with_target(head[0], target_logits.data_ptr(), *head[1:],
                                                     None if device_round is None else device_round.data_ptr(),
                                                     tail[0], tail[1], tnorm.data_ptr(), *tail[2:])
        elif device_round is None:
            st = load().fef_draft_sample(*head, *tail)
        else:
            if device_round.dtype != torch.int32 or device_round.numel() != 1 or device_round.device != dev:
                raise FefError(FEF_ERR_INVALID_ARG, "fef_draft_sample_at_round")
            st = load().fef_draft_sample_at_round(*head, device_round.data_ptr(), *tail)
    if st != FEF_OK:
        raise FefError(st, "fef_draft_sample")
    return out


MASK_TOKEN = -1


def _i32_cuda(t: torch.Tensor, where: str):
    if t.device.type != "cuda" or t.dtype != torch.int32 or not t.is_contiguous():
        raise FefError(FEF_ERR_INVALID_ARG, where)
    return t


def fef_loop_next_window(tokens: torch.Tensor, K: int, stream=None):
    """``tokens [B, L]`` int32 -> ``(window_pos [B, K], row_len [B], unresolved [B])`` (see include/fef.h)."""
    _i32_cuda(tokens, "fef_loop_next_window")
    B, L = tokens.shape
    dev = tokens.device
    with _on(dev, stream):
        window = torch.empty((B, K), dtype=torch.int32, device=dev)
        row_len = torch.empty(B, dtype=torch.int32, device=dev)
        unresolved = torch.empty(B, dtype=torch.int32, device=dev)
        st = load().fef_loop_next_window(tokens.data_ptr(), B, L, K, window.data_ptr(), row_len.data_ptr(),
                                         unresolved.data_ptr(), _stream_ptr(stream))
    if st != FEF_OK:
        raise FefError(st, "fef_loop_next_window")
    return window, row_len, unresolved


def fef_loop_verification_inputs(tokens, window_pos, row_len, draft_tokens, stream=None) -> torch.Tensor:
    """The K verification inputs X^(j_m) of every window, ``[B, K, L]`` int32 (see include/fef.h)."""
    for t in (tokens, window_pos, row_len, draft_tokens):
        _i32_cuda(t, "fef_loop_verification_inputs")
    B, L = tokens.shape
    K = window_pos.shape[1]
    with _on(tokens.device, stream):
        out = torch.empty((B, K, L), dtype=torch.int32, device=tokens.device)
        st = load().fef_loop_verification_inputs(tokens.data_ptr(), window_pos.data_ptr(), row_len.data_ptr(),
                                                 draft_tokens.data_ptr(), B, L, K, out.data_ptr(), _stream_ptr(stream))
    if st != FEF_OK:
        raise FefError(st, "fef_loop_verification_inputs")
    return out


def fef_loop_commit(window_pos, row_len, verified: "VerifyResult", tokens, conf, in_step, stream=None) -> torch.Tensor:
    """Write one verification result back into the loop state (in place); returns ``committed [B]``."""
    for t in (window_pos, row_len, tokens):
        _i32_cuda(t, "fef_loop_commit")
    B, L = tokens.shape
    K = window_pos.shape[1]
    with _on(tokens.device, stream):
        committed = torch.empty(B, dtype=torch.int32, device=tokens.device)
        st = load().fef_loop_commit(window_pos.data_ptr(), row_len.data_ptr(), verified.accept_len.data_ptr(),
                                    verified.tokens.data_ptr(), verified.conf.data_ptr(), B, L, K, tokens.data_ptr(),
                                    conf.data_ptr(), in_step.data_ptr(), committed.data_ptr(), _stream_ptr(stream))
    if st != FEF_OK:
        raise FefError(st, "fef_loop_commit")
    return committed


def fef_loop_advance_round(device_round: torch.Tensor, unresolved: Optional[torch.Tensor] = None, stream=None) -> None:
    """Add one to the device-resident round counter (a one-element int32 CUDA tensor); with
    ``unresolved`` (``[B]`` int32, from ``fef_loop_next_window``) only if some row had work left."""
    _i32_cuda(device_round, "fef_loop_advance_round")
    if unresolved is not None:
        _i32_cuda(unresolved, "fef_loop_advance_round")
    with _on(device_round.device, stream):
        st = load().fef_loop_advance_round(device_round.data_ptr(),
                                           None if unresolved is None else unresolved.data_ptr(),
                                           0 if unresolved is None else unresolved.numel(), _stream_ptr(stream))
    if st != FEF_OK:
        raise FefError(st, "fef_loop_advance_round")


def fef_loop_remask(positions, count, tokens, conf, in_step, stream=None) -> None:
    """Send the selected positions back to MASK and empty the step's set (in place)."""
    B, L = tokens.shape
    k = positions.shape[1]
    with _on(tokens.device, stream):
        st = load().fef_loop_remask(positions.data_ptr() if k else None, count.data_ptr(), B, L, k, tokens.data_ptr(),
                                    conf.data_ptr(), in_step.data_ptr(), _stream_ptr(stream))
    if st != FEF_OK:
        raise FefError(st, "fef_loop_remask")


def fef_remask_select(conf: torch.Tensor, mask: torch.Tensor, k: int, positions: Optional[torch.Tensor] = None,
                      count: Optional[torch.Tensor] = None, stream=None):
    """Enqueue LowConf_k (see ``fef_remask_select`` in include/fef.h).

    ``conf`` ``[B, L]`` float32, ``mask`` ``[B, L]`` uint8 (or bool) ->
    ``(positions [B, k] int32 padded with -1, count [B] int32)``.
    """
    _require_cuda(conf, mask)
    if mask.dtype == torch.bool:
        mask = mask.view(torch.uint8)
    if conf.dim() != 2 or conf.shape != mask.shape or conf.dtype != torch.float32 or mask.dtype != torch.uint8:
        raise FefError(FEF_ERR_INVALID_ARG, "fef_remask_select")
    if not (conf.is_contiguous() and mask.is_contiguous()):
        raise FefError(FEF_ERR_INVALID_ARG, "fef_remask_select")
    B, L = conf.shape
    dev = conf.device
    plain = positions is not None and count is not None and stream is None and torch.cuda.current_device() == dev.index
    with (contextlib.nullcontext() if plain else _on(dev, stream)):
        if positions is None:
            positions = torch.empty((B, max(int(k), 0)), dtype=torch.int32, device=dev)
        if count is None:
            count = torch.empty(B, dtype=torch.int32, device=dev)
        st = load().fef_remask_select(conf.data_ptr(), mask.data_ptr(), B, L, int(k),
                                      positions.data_ptr() if positions.numel() else None,
                                      count.data_ptr(), _stream_ptr(stream))
    if st != FEF_OK:
        raise FefError(st, "fef_remask_select")
    return positions, count


def fef_spec_verify_static(draft_logits: torch.Tensor, target_logits: torch.Tensor, draft_tokens: torch.Tensor,
                           temperature: float, seed: int, step: int, row_len: Optional[torch.Tensor] = None,
                           V: Optional[int] = None, out: Optional[VerifyResult] = None, stream=None) -> VerifyResult:
    """``fef_spec_verify`` without a workspace argument, for callers that must not allocate
    device memory: the scratch is a fixed array inside the library (see
    ``fef_spec_verify_static`` in include/fef.h for the size limit, the first-call set-up
    and the rule that calls sharing a device must not overlap).  ``out`` must be given if
    the caller wants no allocation at all; without it this wrapper allocates the outputs."""
    _require_cuda(draft_logits, target_logits, draft_tokens, row_len)
    if draft_logits.dim() != 3 or draft_logits.shape != target_logits.shape or draft_logits.dtype != target_logits.dtype:
        raise FefError(FEF_ERR_INVALID_ARG, "fef_spec_verify_static")
    if not (draft_logits.is_contiguous() and target_logits.is_contiguous() and draft_tokens.is_contiguous()):
        raise FefError(FEF_ERR_INVALID_ARG, "fef_spec_verify_static")
    if draft_tokens.dtype != torch.int32 or (row_len is not None and row_len.dtype != torch.int32):
        raise FefError(FEF_ERR_INVALID_ARG, "fef_spec_verify_static")
    B, K, ld = draft_logits.shape
    V = ld if V is None else int(V)
    code = _dtype_code(draft_logits)
    dev = draft_logits.device
    # (nothing to allocate and the device already current: no context to enter, which matters for small calls)
    plain = out is not None and workspace is not None and stream is None and torch.cuda.current_device() == dev.index
    with (contextlib.nullcontext() if plain else _on(dev, stream)):
        if out is None:
            out = VerifyResult(torch.empty(B, dtype=torch.int32, device=dev),
                               torch.empty((B, K), dtype=torch.int32, device=dev),
                               torch.empty((B, K), dtype=torch.float32, device=dev),
                               torch.empty(1, dtype=torch.int32, device=dev))
        st = load().fef_spec_verify_static(
            draft_logits.data_ptr(), target_logits.data_ptr(), draft_tokens.data_ptr(),
            None if row_len is None else row_len.data_ptr(), B, K, V, ld, code, float(temperature),
            int(seed) & 0xFFFFFFFFFFFFFFFF, int(step) & 0xFFFFFFFF,
            out.accept_len.data_ptr(), out.tokens.data_ptr(), out.conf.data_ptr(),
            out.device_status.data_ptr(), _stream_ptr(stream))
    if st != FEF_OK:
        raise FefError(st, "fef_spec_verify_static")
    return out


def fef_spec_verify_host_arena_bytes(B: int, K: int, V: int, ld: int, dtype) -> int:
    code = dtype if isinstance(dtype, int) else (FEF_F32 if dtype == torch.float32 else FEF_BF16)
    return int(load().fef_spec_verify_host_arena_bytes(B, K, V, ld, code))


class HostVerifyResult(NamedTuple):
    accept_len: torch.Tensor  # host tensors
    tokens: torch.Tensor
    conf: torch.Tensor
    status: int


def fef_spec_verify_host(draft_logits: torch.Tensor, target_logits: torch.Tensor, draft_tokens: torch.Tensor,
                         temperature: float, seed: int, step: int, arena: torch.Tensor,
                         row_len: Optional[torch.Tensor] = None, V: Optional[int] = None,
                         out: Optional[HostVerifyResult] = None, stream=None) -> HostVerifyResult:
    """Host-buffer form (see ``fef_spec_verify_host`` in include/fef.h): inputs and outputs are
    CPU tensors (pin them for speed), ``arena`` is a CUDA uint8 tensor of at least
    ``fef_spec_verify_host_arena_bytes`` bytes.  Returns after the results are on the host."""
    _require_cuda(arena)
    for t in (draft_logits, target_logits, draft_tokens, row_len):
        if t is not None and (t.device.type != "cpu" or not t.is_contiguous()):
            raise FefError(FEF_ERR_INVALID_ARG, "fef_spec_verify_host")
    B, K, ld = draft_logits.shape
    V = ld if V is None else int(V)
    code = _dtype_code(draft_logits)
    if out is None:
        out = HostVerifyResult(torch.empty(B, dtype=torch.int32).pin_memory(),
                               torch.empty((B, K), dtype=torch.int32).pin_memory(),
                               torch.empty((B, K), dtype=torch.float32).pin_memory(), 0)
    status = ctypes.c_int32(0)
    with _on(arena.device, stream):
        st = load().fef_spec_verify_host(
            draft_logits.data_ptr(), target_logits.data_ptr(), draft_tokens.data_ptr(),
            None if row_len is None else row_len.data_ptr(), B, K, V, ld, code, float(temperature),
            int(seed) & 0xFFFFFFFFFFFFFFFF, int(step) & 0xFFFFFFFF,
            out.accept_len.data_ptr(), out.tokens.data_ptr(), out.conf.data_ptr(), ctypes.byref(status),
            arena.data_ptr(), arena.numel(), _stream_ptr(stream))
    if st != FEF_OK:
        raise FefError(st, "fef_spec_verify_host")
    return HostVerifyResult(out.accept_len, out.tokens, out.conf, int(status.value))


def fef_remask_select_host_arena_bytes(B: int, L: int, k: int) -> int:
    return int(load().fef_remask_select_host_arena_bytes(B, L, k))


def fef_remask_select_host(conf: torch.Tensor, mask: torch.Tensor, k: int, arena: torch.Tensor,
                           positions: Optional[torch.Tensor] = None, count: Optional[torch.Tensor] = None,
                           stream=None):
    """Host-buffer form of ``fef_remask_select``: CPU tensors in and out, staged through ``arena``."""
    _require_cuda(arena)
    if mask.dtype == torch.bool:
        mask = mask.view(torch.uint8)
    if conf.device.type != "cpu" or mask.device.type != "cpu" or conf.shape != mask.shape or conf.dim() != 2:
        raise FefError(FEF_ERR_INVALID_ARG, "fef_remask_select_host")
    B, L = conf.shape
    if positions is None:
        positions = torch.empty((B, max(int(k), 0)), dtype=torch.int32).pin_memory()
    if count is None:
        count = torch.empty(B, dtype=torch.int32).pin_memory()
    with _on(arena.device, stream):
        st = load().fef_remask_select_host(conf.data_ptr(), mask.data_ptr(), B, L, int(k),
                                           positions.data_ptr() if positions.numel() else None, count.data_ptr(),
                                           arena.data_ptr(), arena.numel(), _stream_ptr(stream))
    if st != FEF_OK:
        raise FefError(st, "fef_remask_select_host")
    return positions, count


__all__ = ["fef_loop_advance_round", "fef_loop_next_window", "fef_loop_verification_inputs", "fef_loop_commit", "fef_loop_remask", "MASK_TOKEN",
           "fef_draft_sample", "fef_draft_sample_workspace_bytes", "DraftResult", "fef_spec_verify_static", "HostVerifyResult", "fef_spec_verify_host_arena_bytes", "fef_spec_verify_host",
           "fef_remask_select_host_arena_bytes", "fef_remask_select_host","load", "FefError", "VerifyResult", "fef_status_string", "fef_spec_verify_workspace_bytes",
           "fef_spec_verify", "fef_remask_select", "EXPORTS"]


# ------------------------------------------------------------ verification from hidden states ----
def fef_lmhead_verify_workspace_bytes(B: int, K: int, V: int, d: int) -> int:
    return int(load().fef_lmhead_verify_workspace_bytes(B, K, V, d))


def _bf16_matrix(t: torch.Tensor, where: str):
    if t.device.type != "cuda" or t.dtype != torch.bfloat16 or t.dim() != 2 or not t.is_contiguous():
        raise FefError(FEF_ERR_INVALID_ARG, where)
    return t


def fef_lmhead_verify(draft_hidden: torch.Tensor, target_hidden: torch.Tensor, weight: torch.Tensor,
                      draft_tokens: torch.Tensor, temperature: float, seed: int, step: int,
                      row_len: Optional[torch.Tensor] = None, out: Optional[VerifyResult] = None,
                      workspace: Optional[torch.Tensor] = None, stream=None) -> VerifyResult:
    """Enqueue one verification call on hidden states (see ``fef_lmhead_verify`` in include/fef.h).

    ``draft_hidden`` / ``target_hidden``: ``[B*K, d]`` bfloat16 CUDA tensors; ``weight``: ``[V, d]``
    bfloat16; ``draft_tokens``: ``[B, K]`` int32.
    """
    for t in (draft_hidden, target_hidden, weight):
        _bf16_matrix(t, "fef_lmhead_verify")
    _require_cuda(draft_tokens, row_len)
    if draft_tokens.dtype != torch.int32 or draft_tokens.dim() != 2 or not draft_tokens.is_contiguous():
        raise FefError(FEF_ERR_INVALID_ARG, "fef_lmhead_verify")
    B, K = draft_tokens.shape
    V, d = weight.shape
    if draft_hidden.shape != (B * K, d) or target_hidden.shape != (B * K, d):
        raise FefError(FEF_ERR_INVALID_ARG, "fef_lmhead_verify")
    if row_len is not None and row_len.dtype != torch.int32:
        raise FefError(FEF_ERR_INVALID_ARG, "fef_lmhead_verify")
    dev = weight.device
    with _on(dev, stream):
        if out is None:
            out = VerifyResult(torch.empty(B, dtype=torch.int32, device=dev),
                               torch.empty((B, K), dtype=torch.int32, device=dev),
                               torch.empty((B, K), dtype=torch.float32, device=dev),
                               torch.empty(1, dtype=torch.int32, device=dev))
        if workspace is None:
            workspace = torch.empty(max(fef_lmhead_verify_workspace_bytes(B, K, V, d), 256), dtype=torch.uint8, device=dev)
        st = load().fef_lmhead_verify(draft_hidden.data_ptr(), target_hidden.data_ptr(), weight.data_ptr(),
                                      draft_tokens.data_ptr(), None if row_len is None else row_len.data_ptr(),
                                      B, K, V, d, float(temperature), int(seed) & 0xFFFFFFFFFFFFFFFF,
                                      int(step) & 0xFFFFFFFF, out.accept_len.data_ptr(), out.tokens.data_ptr(),
                                      out.conf.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                      out.device_status.data_ptr(), _stream_ptr(stream))
    if st != FEF_OK:
        raise FefError(st, "fef_lmhead_verify")
    return out


def fef_lmhead_logits(hidden: torch.Tensor, weight: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None):
    """The binary32 logits ``hidden @ weight.T`` as the verification from hidden states sees them
    (see ``fef_lmhead_logits`` in include/fef.h).  Returns ``(logits [rows, ldo] float32, device_status)``;
    the first ``V`` entries of a row are the logits."""
    _bf16_matrix(hidden, "fef_lmhead_logits")
    _bf16_matrix(weight, "fef_lmhead_logits")
    rows, d = hidden.shape
    V = weight.shape[0]
    if weight.shape[1] != d:
        raise FefError(FEF_ERR_INVALID_ARG, "fef_lmhead_logits")
    dev = weight.device
    with _on(dev, stream):
        if out is None:
            out = torch.empty((rows, (V + 3) // 4 * 4), dtype=torch.float32, device=dev)
        status = torch.empty(1, dtype=torch.int32, device=dev)
        st = load().fef_lmhead_logits(hidden.data_ptr(), weight.data_ptr(), rows, V, d, out.data_ptr(), out.shape[1],
                                      status.data_ptr(), _stream_ptr(stream))
    if st != FEF_OK:
        raise FefError(st, "fef_lmhead_logits")
    return out, status


# ---------------------------------------------------------------- device-made logits, whole loop ----
def fef_synth_logits(B: int, K: int, V: int, dtype, draft_std: float, noise_std: float, seed: int, round: int,
                     boost_fraction: float = 0.0, boost: float = 0.0, device_round: Optional[torch.Tensor] = None,
                     out=None, stream=None, device="cuda"):
    """Seeded synthetic (draft_logits, target_logits), ``[B, K, ld]`` with ``ld`` = V rounded up to whole
    16-byte vectors (see ``fef_synth_logits`` in include/fef.h); pass ``V=V`` to the calls that read them."""
    code = FEF_F32 if dtype == torch.float32 else FEF_BF16
    per_vec = 4 if code == FEF_F32 else 8
    ld = (V + per_vec - 1) // per_vec * per_vec
    dev = torch.device(device)
    with _on(dev, stream):
        if out is None:
            out = (torch.empty((B, K, ld), dtype=dtype, device=dev), torch.empty((B, K, ld), dtype=dtype, device=dev))
        st = load().fef_synth_logits(out[0].data_ptr(), out[1].data_ptr(), B, K, V, ld, code, float(draft_std),
                                     float(noise_std), float(boost_fraction), float(boost),
                                     int(seed) & 0xFFFFFFFFFFFFFFFF, int(round) & 0xFFFFFFFF,
                                     None if device_round is None else device_round.data_ptr(), _stream_ptr(stream))
    if st != FEF_OK:
        raise FefError(st, "fef_synth_logits")
    return out


def fef_loop_run_synthetic(B: int, L: int, K: int, V: int, dtype, temperature: float, seed: int, n_steps: int,
                           remask_k: int, draft_std: float, noise_std: float, boost_fraction: float = 0.0,
                           boost: float = 0.0, stream=None, device="cuda"):
    """The whole decoding loop on synthetic logits as one graph launch (see ``fef_loop_run_synthetic`` in
    include/fef.h), from an all-masked state.  Returns dict(tokens, conf, in_step, rounds, device_status)."""
    code = FEF_F32 if dtype == torch.float32 else FEF_BF16
    dev = torch.device(device)
    with _on(dev, stream):
        tokens = torch.full((B, L), MASK_TOKEN, dtype=torch.int32, device=dev)
        conf = torch.full((B, L), -1.0, dtype=torch.float32, device=dev)
        in_step = torch.zeros((B, L), dtype=torch.uint8, device=dev)
        rnd = torch.zeros(1, dtype=torch.int32, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        ws = torch.empty(max(int(load().fef_loop_run_synthetic_workspace_bytes(B, L, K, V, code, remask_k)), 256),
                         dtype=torch.uint8, device=dev)
        st = load().fef_loop_run_synthetic(B, L, K, V, code, float(temperature), int(seed) & 0xFFFFFFFFFFFFFFFF, n_steps,
                                           remask_k, float(draft_std), float(noise_std), float(boost_fraction),
                                           float(boost), tokens.data_ptr(), conf.data_ptr(), in_step.data_ptr(),
                                           rnd.data_ptr(), ws.data_ptr(), ws.numel(), status.data_ptr(), _stream_ptr(stream))
    if st != FEF_OK:
        raise FefError(st, "fef_loop_run_synthetic")
    return dict(tokens=tokens, conf=conf, in_step=in_step, rounds=int(rnd.item()), device_status=int(status.item()))
