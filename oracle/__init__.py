"""Python access to the CPU oracle (test infrastructure, not the product).

Builds ``oracle/fef_oracle.cpp`` with g++ into ``oracle/libfef_oracle.so`` on
first use and exposes its C entry points on host arrays.  Only tests, the smoke
check and the benchmark's CPU-baseline leg import this module; it shares no
code with the CUDA library and never imports it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fef_oracle.cpp")
_HDR = os.path.join(_HERE, "fef_oracle.h")
_LIB = os.path.join(_HERE, "libfef_oracle.so")

OK, ERR_INVALID_ARG, ERR_DTYPE, ERR_NONFINITE, ERR_TOKEN_RANGE = 0, 1, 2, 7, 8
F32, BF16, F64 = 0, 1, 2

_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (plain ``g++ -O2``, single-threaded code)."""
    newest_src = max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest_src:
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(
            ["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-Wall", "-Wextra", "-o", tmp, _SRC]
        )
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    with _lock:
        if _lib is None:
            L = ctypes.CDLL(build())
            vp, i32, i64, u32, u64, f32 = (
                ctypes.c_void_p,
                ctypes.c_int,
                ctypes.c_int64,
                ctypes.c_uint32,
                ctypes.c_uint64,
                ctypes.c_float,
            )
            L.fef_oracle_philox4x32_10.argtypes = [vp, vp, vp]
            L.fef_oracle_philox4x32_10.restype = None
            L.fef_oracle_uniform.argtypes = [u64, u32, u32, u32, u32, u32, u32]
            L.fef_oracle_uniform.restype = ctypes.c_double
            L.fef_oracle_row_laws.argtypes = [vp, vp, i32, i32, f32, vp, vp, vp, vp]
            L.fef_oracle_row_laws.restype = i32
            L.fef_oracle_spec_verify.argtypes = [
                vp, vp, vp, vp, i32, i32, i32, i64, i32, f32, u64, u32, u32, vp, vp, vp, vp, vp,
            ]
            L.fef_oracle_spec_verify.restype = i32
            L.fef_oracle_draft_sample.argtypes = [vp, vp, i32, i32, i32, i64, i32, f32, u64, u32, u32, vp, vp]
            L.fef_oracle_draft_sample.restype = i32
            L.fef_oracle_remask_select.argtypes = [vp, vp, i32, i32, i32, vp, vp]
            L.fef_oracle_remask_select.restype = i32
            _lib = L
    return _lib


def _logits_as_numpy(x):
    """Return (contiguous numpy array viewing the raw storage, dtype code)."""
    try:
        import torch
    except ImportError:  # pragma: no cover
        torch = None
    if torch is not None and isinstance(x, torch.Tensor):
        if x.device.type != "cpu":
            raise ValueError("the oracle takes host tensors")
        x = x.contiguous()
        if x.dtype == torch.bfloat16:
            return x.view(torch.int16).numpy().view(np.uint16), BF16
        if x.dtype == torch.float32:
            return x.numpy(), F32
        if x.dtype == torch.float64:
            return x.numpy(), F64
        raise ValueError("logits must be float32 or bfloat16")
    x = np.ascontiguousarray(x)
    if x.dtype == np.float64:
        return x, F64
    if x.dtype == np.float32:
        return x, F32
    if x.dtype == np.uint16:  # raw bfloat16 bit patterns
        return x, BF16
    raise ValueError("logits must be float32, or uint16 holding bfloat16 bits")


def _i32(x):
    try:
        import torch

        if isinstance(x, torch.Tensor):
            x = x.cpu().numpy()
    except ImportError:  # pragma: no cover
        pass
    return np.ascontiguousarray(x, dtype=np.int32)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def philox4x32_10(ctr, key):
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().fef_oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def uniform(seed, stream, j, b, pos, step, lane):
    return lib().fef_oracle_uniform(seed, stream, j, b, pos, step, lane)


def row_laws(p_logits, q_logits, temperature=1.0):
    """(pi, rho, resid, alpha) of one position; float64 arrays of length V."""
    p, dt = _logits_as_numpy(p_logits)
    q, dt2 = _logits_as_numpy(q_logits)
    assert dt == dt2 and p.shape == q.shape and p.ndim == 1
    V = p.shape[0]
    pi, rho, res = (np.zeros(V), np.zeros(V), np.zeros(V))
    alpha = np.zeros(1)
    st = lib().fef_oracle_row_laws(_ptr(p), _ptr(q), V, dt, temperature, _ptr(pi), _ptr(rho), _ptr(res), _ptr(alpha))
    if st != OK:
        raise ValueError("fef_oracle_row_laws status %d" % st)
    return pi, rho, res, float(alpha[0])


def spec_verify(draft_logits, target_logits, draft_tokens, temperature, seed, step, row_len=None, V=None,
                batch_offset=0):
    """Run one verification call.  Logits are [B, K, ld]; ``V`` defaults to ld;
    window b uses the random numbers of batch row ``batch_offset + b``.

    Returns a dict: status, accept_len [B], tokens [B,K], conf [B,K] (float64),
    accept_margin [B,K], gumbel_gap [B].
    """
    q, dt = _logits_as_numpy(draft_logits)
    p, dt2 = _logits_as_numpy(target_logits)
    assert dt == dt2 and q.shape == p.shape and q.ndim == 3
    B, K, ld = q.shape
    V = ld if V is None else V
    tok = _i32(draft_tokens).reshape(B, K)
    rl = None if row_len is None else _i32(row_len).reshape(B)
    accept_len = np.zeros(B, dtype=np.int32)
    tokens = np.zeros((B, K), dtype=np.int32)
    conf = np.zeros((B, K), dtype=np.float64)
    margin = np.zeros((B, K), dtype=np.float64)
    gap = np.zeros(B, dtype=np.float64)
    st = lib().fef_oracle_spec_verify(
        _ptr(q), _ptr(p), _ptr(tok), _ptr(rl), B, K, V, ld, dt, temperature, seed, step, batch_offset,
        _ptr(accept_len), _ptr(tokens), _ptr(conf), _ptr(margin), _ptr(gap),
    )
    return dict(status=st, accept_len=accept_len, tokens=tokens, conf=conf, accept_margin=margin, gumbel_gap=gap)


def draft_sample(draft_logits, temperature, seed, step, row_len=None, V=None, batch_offset=0):
    """Draw the draft tokens of one call.  Logits are [B, K, ld]; ``V`` defaults to ld.

    Returns a dict: status, tokens [B,K] (int32, -1 where nothing was drawn), gumbel_gap [B,K].
    """
    q, dt = _logits_as_numpy(draft_logits)
    assert q.ndim == 3
    B, K, ld = q.shape
    V = ld if V is None else V
    rl = None if row_len is None else _i32(row_len).reshape(B)
    tokens = np.zeros((B, K), dtype=np.int32)
    gap = np.zeros((B, K), dtype=np.float64)
    st = lib().fef_oracle_draft_sample(_ptr(q), _ptr(rl), B, K, V, ld, dt, temperature, seed, step, batch_offset,
                                       _ptr(tokens), _ptr(gap))
    return dict(status=st, tokens=tokens, gumbel_gap=gap)


def remask_select(conf, mask, k):
    """LowConf_k per batch row: (positions [B,k] int32 padded with -1, count [B])."""
    try:
        import torch

        if isinstance(conf, torch.Tensor):
            conf = conf.cpu().numpy()
        if isinstance(mask, torch.Tensor):
            mask = mask.cpu().numpy()
    except ImportError:  # pragma: no cover
        pass
    c = np.ascontiguousarray(conf, dtype=np.float32)
    m = np.ascontiguousarray(mask, dtype=np.uint8)
    assert c.ndim == 2 and c.shape == m.shape
    B, L = c.shape
    pos = np.zeros((B, max(k, 0)), dtype=np.int32)
    cnt = np.zeros(B, dtype=np.int32)
    st = lib().fef_oracle_remask_select(_ptr(c), _ptr(m), B, L, k, _ptr(pos), _ptr(cnt))
    if st != OK:
        raise ValueError("fef_oracle_remask_select status %d" % st)
    return pos, cnt
