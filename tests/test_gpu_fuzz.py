"""Seeded random shapes and contents against the CPU oracle: window counts, window lengths,
vocabulary sizes, paddings, temperatures, partial windows and -inf patterns that the hand-picked
cases do not list (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
from oracle.compare import ParityReport, compare_verify
from paper_2605_14305_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fef():
    import paper_2605_14305_b200 as lib

    lib.load(build_if_missing=True)
    return lib


def _random_config(rng):
    kind = rng.integers(0, 4)
    if kind == 0:      # many short rows (the warp-per-row kernel when there are enough of them)
        B, K, V = int(rng.integers(20, 90)), int(rng.integers(8, 65)), int(rng.integers(1, 3000))
    elif kind == 1:    # few long rows (many claims per row)
        B, K, V = int(rng.integers(1, 4)), int(rng.integers(1, 9)), int(rng.integers(20000, 90000))
    elif kind == 2:    # tiny everything
        B, K, V = int(rng.integers(1, 6)), int(rng.integers(1, 6)), int(rng.integers(1, 40))
    else:
        B, K, V = int(rng.integers(1, 30)), int(rng.integers(1, 65)), int(rng.integers(100, 12000))
    dtype = torch.bfloat16 if rng.integers(0, 2) else torch.float32
    T = float(rng.choice([0.0, 0.5, 1.0, 2.0]))
    pad = int(rng.integers(0, 3)) * 8
    ld = -(-V // 8) * 8 + pad
    return B, K, V, ld, dtype, T


@pytest.mark.parametrize("chunk", range(12))
def test_random_calls_match_the_oracle(fef, chunk):
    rng = np.random.default_rng(9000 + chunk)
    total = ParityReport()
    for case in range(25):
        B, K, V, ld, dtype, T = _random_config(rng)
        g = torch.Generator(device="cuda").manual_seed(int(rng.integers(1, 1 << 30)))
        scale = float(rng.choice([0.5, 2.0, 6.0]))
        q = torch.randn((B, K, ld), generator=g, device="cuda") * scale
        p = q + torch.randn((B, K, ld), generator=g, device="cuda") * float(rng.choice([0.0, 0.3, 1.0, 3.0]))
        if rng.integers(0, 3) == 0:          # a random share of the vocabulary without mass, per tensor
            q = torch.where(torch.rand((B, K, ld), generator=g, device="cuda") < 0.3, float("-inf"), q)
            p = torch.where(torch.rand((B, K, ld), generator=g, device="cuda") < 0.3, float("-inf"), p)
            q[:, :, 0] = 0.0                  # every row keeps one finite entry
            p[:, :, 0] = 0.0
        q, p = q.to(dtype), p.to(dtype)
        if ld > V:                            # padding must never be read
            q[:, :, V:] = float("nan")
            p[:, :, V:] = float("inf")
        tok = synth.sample_draft_tokens(q[:, :, :V].contiguous(), max(T, 0.5), int(rng.integers(1, 1 << 30)))
        if T == 0.0:                          # let some windows get past position 0
            top = p[:, :, :V].float().argmax(-1).to(torch.int32)
            tok = torch.where(torch.rand(tok.shape, device="cuda") < 0.5, tok, top)
        row_len = None
        if rng.integers(0, 2):
            row_len = torch.as_tensor(rng.integers(0, K + 1, size=B).astype(np.int32), device="cuda")
        seed, step = int(rng.integers(0, 1 << 62)), int(rng.integers(0, 1 << 31))
        r = fef.fef_spec_verify(q, p, tok, T, seed, step, row_len=row_len, V=V)
        torch.cuda.synchronize()
        ref = oracle.spec_verify(q.cpu(), p.cpu(), tok.cpu(), T, seed, step,
                                 row_len=None if row_len is None else row_len.cpu(), V=V)
        assert ref["status"] == 0 and int(r.device_status.item()) == 0, (B, K, V, ld, dtype, T)
        rep = compare_verify(r.accept_len.cpu().numpy(), r.tokens.cpu().numpy(), r.conf.cpu().numpy(), ref)
        assert rep.ok, ((B, K, V, ld, dtype, T), rep.mismatches[:5])
        total.merge(rep)
        if T > 0 and case % 4 == 0:           # the draft draws of the same rows
            d = fef.fef_draft_sample(q, T, seed, step, row_len=row_len, V=V)
            od = oracle.draft_sample(q.cpu(), T, seed, step, row_len=None if row_len is None else row_len.cpu(), V=V)
            n = np.full(B, K) if row_len is None else row_len.cpu().numpy()
            used = np.arange(K)[None, :] < n[:, None]
            sure = od["gumbel_gap"] > 1e-6
            assert (d.tokens.cpu().numpy()[used & sure] == od["tokens"][used & sure]).all(), (B, K, V, ld, dtype, T)
    print(total.summary())
    assert total.within_budget


def test_random_low_confidence_selections_match_the_oracle(fef):
    rng = np.random.default_rng(4242)
    for case in range(80):
        B, L = int(rng.integers(1, 70)), int(rng.integers(1, 2200))
        k = int(rng.integers(0, min(L, 300) + 1))
        conf = rng.random((B, L)).astype(np.float32)
        if case % 3 == 0:      # many ties
            conf = np.round(conf * 4) / 4
        if case % 5 == 0:      # signed zeros and NaNs
            conf[rng.random((B, L)) < 0.05] = -0.0
            conf[rng.random((B, L)) < 0.02] = np.nan
        mask = (rng.random((B, L)) < rng.choice([0.0, 0.1, 0.6, 1.0])).astype(np.uint8)
        pos, cnt = fef.fef_remask_select(torch.as_tensor(conf).cuda(), torch.as_tensor(mask).cuda(), k)
        opos, ocnt = oracle.remask_select(conf, mask, k)
        assert (cnt.cpu().numpy() == ocnt).all(), (B, L, k)
        assert (pos.cpu().numpy() == opos).all(), (B, L, k)
