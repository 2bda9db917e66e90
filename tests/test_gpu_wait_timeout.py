"""A bounded wait of the streaming kernel running out (needs a B200).

Every wait inside the kernels is bounded; when one runs out the kernel must report FEF_ERR_TIMEOUT,
let what is in flight land, return, and leave the context usable.  This is exercised with a test
build of the library (-DFEF_TEST_HOOKS, see _build.build_test_hooks) in which the streaming
kernel's first CTA can be told to withhold one stage of its ring - a stage for which no copy was
issued - with a wait limit of a few milliseconds.  Nothing faults, traps or hangs: the consumers'
wait for that stage simply ends after the limit."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from oracle.compare import compare_verify

pytestmark = pytest.mark.gpu

FEF_ERR_TIMEOUT = 6


def _load_hooks_library():
    from paper_2605_14305_b200 import _build

    L = ctypes.CDLL(_build.build_test_hooks())
    vp, i32, i64, u32, u64, f32, sz = (ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_uint32,
                                       ctypes.c_uint64, ctypes.c_float, ctypes.c_size_t)
    L.fef_spec_verify_workspace_bytes.argtypes = [i32, i32, i32, i32]
    L.fef_spec_verify_workspace_bytes.restype = sz
    L.fef_spec_verify.argtypes = [vp, vp, vp, vp, i32, i32, i32, i64, i32, f32, u64, u32, vp, vp, vp, vp, sz, vp, vp]
    L.fef_spec_verify.restype = i32
    L.fef_test_withhold_stage_once.argtypes = [i32, u64]
    L.fef_test_withhold_stage_once.restype = None
    return L


@pytest.mark.parametrize("T", [1.0, 0.0])
def test_a_wait_that_runs_out_reports_timeout_and_the_next_call_is_exact(T):
    L = _load_hooks_library()
    B, K, V = 8, 32, 50000   # (large enough for the streaming kernel in sampling mode too)
    g = torch.Generator(device="cuda").manual_seed(3)
    q = (torch.randn((B, K, V), generator=g, device="cuda") * 2).to(torch.bfloat16)
    p = (q.float() + torch.randn((B, K, V), generator=g, device="cuda") * 0.7).to(torch.bfloat16)
    tok = torch.randint(0, V, (B, K), generator=g, device="cuda", dtype=torch.int32)
    ws = torch.zeros(int(L.fef_spec_verify_workspace_bytes(B, K, V, 1)), dtype=torch.uint8, device="cuda")
    accept = torch.full((B,), 77, dtype=torch.int32, device="cuda")
    tokens = torch.full((B, K), 77, dtype=torch.int32, device="cuda")
    conf = torch.full((B, K), 77.0, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream

    def call(step):
        return L.fef_spec_verify(q.data_ptr(), p.data_ptr(), tok.data_ptr(), None, B, K, V, V, 1, T, 5, step,
                                 accept.data_ptr(), tokens.data_ptr(), conf.data_ptr(), ws.data_ptr(), ws.numel(),
                                 status.data_ptr(), stream)

    # the first CTA's producer delivers one stage and withholds the next; waits give up after 3 ms
    L.fef_test_withhold_stage_once(1, 3_000_000)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    assert call(1) == 0
    t1.record()
    torch.cuda.synchronize()                      # the kernels returned: nothing hangs
    assert int(status.item()) == FEF_ERR_TIMEOUT
    assert t0.elapsed_time(t1) < 500.0            # the limit, not the one-second default, ended the wait
    assert (accept.cpu().numpy() == -1).all()     # no window is decided from incomplete sums
    assert (tokens.cpu().numpy() == -1).all() and (conf.cpu().numpy() == -1.0).all()

    # the next ordinary call on the same stream and scratch is exact
    assert call(2) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle.spec_verify(q.cpu(), p.cpu(), tok.cpu(), T, 5, 2)
    rep = compare_verify(accept.cpu().numpy(), tokens.cpu().numpy(), conf.cpu().numpy(), ref)
    assert rep.ok, rep.mismatches

