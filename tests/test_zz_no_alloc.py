"""fef_spec_verify_static: the entry point for callers that may not allocate device memory.

Some programs that embed this library cannot call cudaMalloc where they verify: they run
inside a memory plan that someone else owns (a server that carved up the whole device at
start-up), or on a path where an allocation's implicit synchronisation is unacceptable.
For them the scratch lives in a fixed array inside the library.  This test drives that
entry point through the C ABI twice in a row on different inputs and sizes and checks
each result against fef_spec_verify with a caller-provided workspace (the integers must
be identical and the confidences must agree to the tolerance the other GPU tests use)
and, directly, against the CPU oracle.
The second call also shows that what the first call left in the shared scratch does not
leak into later results.  Collected last on purpose (file name), so a run that stops at
the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

CONF_RTOL = 1e-5


def _case(B, K, V, dtype, seed):
    from paper_2605_14305_b200 import synth

    w = synth.LLADA_BATCHED.with_(B=B, K=K, V=V, dtype=dtype, noise_std=0.6)
    return synth.make_call(w, seed=seed, device="cuda")


def _matches_oracle(got, q, p, tok, T, seed, step, row_len=None):
    import oracle
    from oracle.compare import compare_verify

    ref = oracle.spec_verify(q.cpu(), p.cpu(), tok.cpu(), T, seed, step, row_len=None if row_len is None else row_len.cpu())
    rep = compare_verify(got.accept_len.cpu().numpy(), got.tokens.cpu().numpy(), got.conf.cpu().numpy(), ref)
    assert rep.ok and rep.excused == 0, rep.mismatches[:5]


def _same(a, b):
    assert (a.accept_len.cpu().numpy() == b.accept_len.cpu().numpy()).all()
    assert (a.tokens.cpu().numpy() == b.tokens.cpu().numpy()).all()
    ca, cb = a.conf.cpu().numpy().astype(np.float64), b.conf.cpu().numpy().astype(np.float64)
    assert (np.abs(ca - cb) <= CONF_RTOL * np.abs(cb)).all()
    assert int(a.device_status.item()) == int(b.device_status.item()) == 0


def test_static_scratch_entry_point_matches_workspace_entry_point_twice_in_a_row():
    import paper_2605_14305_b200 as fef

    fef.load(build_if_missing=True)
    # first call: a shape that spreads every row over several CTAs and rejects in most windows
    q, p, tok = _case(16, 32, 126464, torch.bfloat16, seed=1)
    want = fef.fef_spec_verify(q, p, tok, 0.7, seed=5, step=1)
    got = fef.fef_spec_verify_static(q, p, tok, 0.7, seed=5, step=1)
    torch.cuda.synchronize()
    _same(got, want)
    _matches_oracle(got, q, p, tok, 0.7, 5, 1)
    assert (want.accept_len.cpu().numpy() < 32).any()  # the residual path ran

    # second call right after it: other sizes, other dtype, a ragged row length, fewer windows,
    # so stale partials, tasks and candidates of the first call sit in the scratch
    q, p, tok = _case(5, 7, 4100, torch.float32, seed=2)
    row_len = torch.tensor([7, 0, 3, 7, 1], dtype=torch.int32, device="cuda")
    want = fef.fef_spec_verify(q, p, tok, 1.0, seed=6, step=2, row_len=row_len)
    got = fef.fef_spec_verify_static(q, p, tok, 1.0, seed=6, step=2, row_len=row_len)
    torch.cuda.synchronize()
    _same(got, want)
    _matches_oracle(got, q, p, tok, 1.0, 6, 2, row_len=row_len)

    # and the greedy mode through the same scratch
    want = fef.fef_spec_verify(q, p, tok, 0.0, seed=6, step=3)
    got = fef.fef_spec_verify_static(q, p, tok, 0.0, seed=6, step=3)
    torch.cuda.synchronize()
    _same(got, want)
    _matches_oracle(got, q, p, tok, 0.0, 6, 3)


def test_static_scratch_entry_point_refuses_sizes_beyond_its_buffer():
    import paper_2605_14305_b200 as fef

    fef.load(build_if_missing=True)
    B, K, V = 4096, 64, 64  # small in bytes of logits, but far more windows than the buffer covers
    assert fef.fef_spec_verify_workspace_bytes(B, K, V, torch.float32) > fef.FEF_STATIC_SCRATCH_BYTES
    q = torch.zeros((B, K, V), device="cuda")
    tok = torch.zeros((B, K), dtype=torch.int32, device="cuda")
    with pytest.raises(fef.FefError) as err:
        fef.fef_spec_verify_static(q, q, tok, 1.0, seed=0, step=0)
    assert err.value.status == fef.FEF_ERR_TOO_LARGE
    assert "scratch" in str(err.value)
