"""Vocabulary-parallel verification (slices of the vocabulary on different ranks) against the CPU
oracle on the full rows.  The ranks are emulated one after the other on a single GPU (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
from oracle.compare import compare_verify
from paper_2605_14305_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fef():
    import paper_2605_14305_b200 as lib

    lib.load(build_if_missing=True)
    return lib


def _slices(q, p, ranks):
    from paper_2605_14305_b200.vocab_parallel import shard_vocab

    V = q.shape[2]
    out = []
    for off, width in shard_vocab(V, ranks):
        ld = -(-width // 8) * 8
        qs = torch.full(q.shape[:2] + (ld,), float("nan"), dtype=q.dtype, device=q.device)  # padding must never be read
        ps = torch.full_like(qs, float("inf"))
        qs[:, :, :width] = q[:, :, off:off + width]
        ps[:, :, :width] = p[:, :, off:off + width]
        out.append((qs.contiguous(), ps.contiguous(), off, width))
    return out


def _run(fef, q, p, tok, T, seed, step, ranks, row_len=None, expect_status=0):
    from paper_2605_14305_b200.vocab_parallel import fef_spec_verify_sharded_on_one_device

    V = q.shape[2]
    outs = fef_spec_verify_sharded_on_one_device(_slices(q, p, ranks), tok, T, seed, step, V, row_len=row_len)
    torch.cuda.synchronize()
    first = outs[0]
    for o in outs[1:]:  # every rank decides the same
        assert (o.accept_len == first.accept_len).all() and (o.tokens == first.tokens).all()
        assert (o.conf == first.conf).all()
    ref = oracle.spec_verify(q.cpu(), p.cpu(), tok.cpu(), T, seed, step, row_len=None if row_len is None else row_len.cpu())
    assert ref["status"] == expect_status
    assert max(int(o.device_status.item()) for o in outs) == expect_status
    rep = compare_verify(first.accept_len.cpu().numpy(), first.tokens.cpu().numpy(), first.conf.cpu().numpy(), ref)
    assert rep.ok, rep.mismatches[:5]
    return first, rep


def _case(B, K, V, dtype, noise, seed, scale=2.0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    q = (torch.randn((B, K, V), generator=g, device="cuda") * scale)
    p = q + torch.randn((B, K, V), generator=g, device="cuda") * noise
    q, p = q.to(dtype).contiguous(), p.to(dtype).contiguous()
    tok = synth.sample_draft_tokens(q, 1.0, seed + 1)
    return q, p, tok


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("B,K,V,ranks", [(1, 1, 16, 2), (2, 3, 40, 2), (3, 4, 1000, 3), (2, 8, 4097, 4), (5, 4, 33, 4),
                                         (4, 32, 9000, 8), (2, 64, 70001, 3), (6, 5, 2048, 1),
                                         (40, 32, 2000, 2)])  # the last: short slices, many rows (warp per row)
def test_sharded_verification_matches_the_oracle_on_the_full_rows(fef, dtype, B, K, V, ranks):
    q, p, tok = _case(B, K, V, dtype, 0.6, seed=B * 100 + K + V)
    for T, step in ((1.0, 3), (0.7, 4)):
        out, _ = _run(fef, q, p, tok, T, 11, step, ranks)
        ld = -(-V // 8) * 8                                   # and the single-GPU call on the same rows
        qp = torch.zeros((B, K, ld), dtype=dtype, device="cuda")
        pp = torch.zeros_like(qp)
        qp[:, :, :V], pp[:, :, :V] = q, p
        plain = fef.fef_spec_verify(qp, pp, tok, T, 11, step, V=V)
        assert (plain.accept_len == out.accept_len).all() and (plain.tokens == out.tokens).all()
        assert torch.allclose(plain.conf, out.conf, rtol=1e-5, atol=0)


def test_sharded_llada_shape_sampled_windows(fef):
    w = synth.HEADLINE.with_(B=8, K=32, noise_std=0.7)
    q, p = synth.make_logits(w, seed=77, device="cuda")
    tok = synth.sample_draft_tokens(q, w.temperature, 78)
    out, rep = _run(fef, q, p, tok, w.temperature, 5, 9, ranks=4)
    assert rep.windows == 8
    print(rep.summary())


def test_sharded_row_len_identical_laws_and_minus_inf(fef):
    q, p, tok = _case(4, 8, 520, torch.float32, 0.5, seed=5)
    rl = torch.tensor([8, 0, 3, 1], dtype=torch.int32, device="cuda")
    out, _ = _run(fef, q, p, tok, 1.0, 2, 1, ranks=3, row_len=rl)
    assert int(out.accept_len[1].item()) == 0
    out, _ = _run(fef, q, q.clone(), tok, 1.0, 2, 2, ranks=2)          # p = q: everything is accepted
    assert (out.accept_len == 8).all()
    q2, p2 = q.clone(), p.clone()
    q2[:, :, 100:300] = float("-inf")                                   # a whole slice region without mass
    p2[:, :, 250:400] = float("-inf")
    tok2 = synth.sample_draft_tokens(q2, 1.0, 9)
    _run(fef, q2, p2, tok2, 1.0, 2, 3, ranks=4)
    q3 = q.clone()
    q3[:, :, :176] = float("-inf")                                      # rank 0 of 3 holds no draft mass at all
    tok3 = synth.sample_draft_tokens(q3, 1.0, 10)
    _run(fef, q3, p, tok3, 1.0, 2, 4, ranks=3)


def test_sharded_data_errors(fef):
    q, p, tok = _case(3, 4, 264, torch.float32, 0.5, seed=6)
    bad = p.clone()
    bad[1, 2, 200] = float("nan")                                       # lives in the last of three slices
    out, _ = _run(fef, q, bad, tok, 1.0, 2, 1, ranks=3, expect_status=fef.FEF_ERR_NONFINITE)
    assert int(out.accept_len[1].item()) == -1 and int(out.accept_len[0].item()) >= 0
    t2 = tok.clone()
    t2[2, 0] = 264                                                      # one past the vocabulary
    out, _ = _run(fef, q, p, t2, 1.0, 2, 1, ranks=2, expect_status=fef.FEF_ERR_TOKEN_RANGE)
    assert int(out.accept_len[2].item()) == -1


def test_sharded_argument_errors(fef):
    from paper_2605_14305_b200.vocab_parallel import fef_spec_verify_sharded_on_one_device, shard_vocab

    q, p, tok = _case(2, 2, 64, torch.float32, 0.5, seed=7)
    with pytest.raises(fef.FefError):   # offsets must be multiples of 8
        fef_spec_verify_sharded_on_one_device([(q[:, :, :32].contiguous(), p[:, :, :32].contiguous(), 0),
                                               (q[:, :, 32:].contiguous(), p[:, :, 32:].contiguous(), 36)], tok, 1.0, 1, 1, 64)
    with pytest.raises(fef.FefError):   # sampling mode only
        fef_spec_verify_sharded_on_one_device(_slices(q, p, 2), tok, 0.0, 1, 1, 64)
    assert shard_vocab(126464, 8)[0] == (0, 15808) and sum(w for _, w in shard_vocab(70001, 3)) == 70001


@pytest.mark.parametrize("chunk", range(4))
def test_sharded_random_calls_match_the_oracle(fef, chunk):
    rng = np.random.default_rng(500 + chunk)
    for case in range(12):
        B, K = int(rng.integers(1, 50)), int(rng.integers(1, 65))
        V = int(rng.integers(16, 6000))
        ranks = int(rng.integers(1, min(8, V // 8) + 1))
        dtype = torch.bfloat16 if rng.integers(0, 2) else torch.float32
        T = float(rng.choice([0.5, 1.0, 2.0]))
        q, p, tok = _case(B, K, V, dtype, float(rng.choice([0.0, 0.4, 1.5])), seed=int(rng.integers(1, 1 << 30)),
                          scale=float(rng.choice([0.5, 2.0, 5.0])))
        if rng.integers(0, 3) == 0:
            g = torch.Generator(device="cuda").manual_seed(case + 1)
            q = torch.where(torch.rand(q.shape, generator=g, device="cuda") < 0.3, float("-inf"), q.float()).to(dtype)
            p = torch.where(torch.rand(p.shape, generator=g, device="cuda") < 0.3, float("-inf"), p.float()).to(dtype)
            q[:, :, 0], p[:, :, 0] = 0.0, 0.0
            tok = synth.sample_draft_tokens(q, 1.0, case + 3)
        rl = None
        if rng.integers(0, 2):
            rl = torch.as_tensor(rng.integers(0, K + 1, size=B).astype(np.int32), device="cuda")
        _run(fef, q, p, tok, T, int(rng.integers(0, 1 << 62)), int(rng.integers(0, 1 << 31)), ranks, row_len=rl)
