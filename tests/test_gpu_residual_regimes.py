"""The residual draw where the two laws nearly coincide (needs a B200).

With pi close to rho the numerator [pi - rho]_+ of the residual law is a small difference of two
nearly equal numbers, so any error in the laws' normalisers or in binary32 arithmetic is
amplified by pi / (pi - rho).  These cases force a rejection at position 0 of every window (the
draft token gets target probability zero, or next to zero) with a residual mass from about 1e-7 to
1e-2, and compare the replacement token with the oracle's: every draw outside the 1e-6 margins must
agree."""
import math

import numpy as np
import pytest
import torch

import oracle
from oracle.compare import ParityReport, compare_verify

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fef():
    import paper_2605_14305_b200 as lib

    lib.load(build_if_missing=True)
    return lib


def _draft_rows(B, V, dtype, seed, peaked):
    g = torch.Generator(device="cuda").manual_seed(seed)
    q = torch.randn((B, 1, V), generator=g, device="cuda") * 2.0
    if peaked:
        q = q + 8.0 * (torch.rand((B, 1, V), generator=g, device="cuda") < 0.01)
    return q.to(dtype), g


def _token_with_mass(q, mass):
    """Per row the vocabulary id whose draft probability is closest to `mass` (on a log scale)."""
    logp = torch.log_softmax(q.float()[:, 0, :], dim=-1)
    return (logp - math.log(mass)).abs().argmin(dim=-1).to(torch.int32).view(-1, 1)


def _run(fef, q, p, tok, T, seed, step):
    r = fef.fef_spec_verify(q, p, tok, T, seed, step)
    torch.cuda.synchronize()
    assert int(r.device_status.item()) == 0
    ref = oracle.spec_verify(q.cpu(), p.cpu(), tok.cpu(), T, seed, step)
    assert ref["status"] == 0
    rep = compare_verify(r.accept_len.cpu().numpy(), r.tokens.cpu().numpy(), r.conf.cpu().numpy(), ref)
    assert rep.ok, rep.mismatches[:5]
    return rep, ref


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V,B", [(1000, 160), (8192, 120), (32000, 80), (126464, 48)])
def test_target_equals_draft_except_at_the_draft_token(fef, dtype, V, B):
    """pi = rho renormalised without the draft token: r_x = rho_x * eta for every other x with one
    common eta ~ rho(token), from 1e-7 to 1e-2."""
    total = ParityReport()
    rejected = 0
    for n, mass in enumerate((1e-7, 1e-6, 1e-5, 1e-4, 1e-3, 1e-2)):
        for lowered in (float("-inf"), -25.0):
            q, _ = _draft_rows(B, V, dtype, 400 + n, peaked=(n % 2 == 0))
            tok = _token_with_mass(q, mass)
            p = q.clone()
            idx = tok.long().view(B, 1, 1)
            if lowered == float("-inf"):
                p.scatter_(2, idx, float("-inf"))
            else:
                p.scatter_(2, idx, (q.gather(2, idx).float() + lowered).to(dtype))
            rep, ref = _run(fef, q, p, tok, 1.0, 31 + n, 7 * n + (lowered != float("-inf")))
            rejected += int((ref["accept_len"] == 0).sum())
            total.merge(rep)
    print(total.summary(), "forced rejections", rejected)
    assert rejected >= 0.98 * 12 * B
    assert total.within_budget


@pytest.mark.parametrize("sigma", [1e-4, 1e-3, 1e-2])
@pytest.mark.parametrize("V,B", [(1000, 120), (32000, 60), (126464, 40)])
def test_target_is_draft_plus_small_noise(fef, sigma, V, B):
    """target = draft + N(0, sigma^2) in binary32 (bfloat16 would round the noise away), the draft
    token's target logit at -inf so that position 0 rejects; the token's mass is chosen around
    sigma, where the renormalisation and the noise contribute alike."""
    total = ParityReport()
    rejected = 0
    for n, mass in enumerate((1e-6, 1e-4, 1e-2)):
        for T in (1.0, 0.7):
            q, g = _draft_rows(B, V, torch.float32, 900 + n, peaked=True)
            p = q + torch.randn(q.shape, generator=g, device="cuda") * sigma
            tok = _token_with_mass(q / T, mass)
            p.scatter_(2, tok.long().view(B, 1, 1), float("-inf"))
            rep, ref = _run(fef, q, p, tok, T, 77 + n, 3 * n + int(T < 1))
            rejected += int((ref["accept_len"] == 0).sum())
            total.merge(rep)
    print(total.summary(), "forced rejections", rejected)
    assert rejected == 6 * B
    assert total.within_budget


def test_small_noise_in_bfloat16_and_a_common_shift(fef):
    """bfloat16 rounds most of the noise away (many ids with pi = rho exactly, a few one step apart);
    a large common offset between the tensors cancels in the laws but not in the logits."""
    total = ParityReport()
    for n, (dtype, sigma, shift) in enumerate([(torch.bfloat16, 1e-2, 0.0), (torch.bfloat16, 3e-2, 0.0),
                                               (torch.float32, 1e-3, 300.0), (torch.float32, 1e-2, -700.0)]):
        B, V = 64, 50000
        q, g = _draft_rows(B, V, dtype, 1300 + n, peaked=True)
        p = (q.float() + torch.randn(q.shape, generator=g, device="cuda") * sigma + shift).to(dtype)
        tok = _token_with_mass(q, 1e-3)
        p.scatter_(2, tok.long().view(B, 1, 1), float("-inf"))
        rep, ref = _run(fef, q, p, tok, 1.0, 5 + n, n)
        assert (ref["accept_len"] == 0).all()
        total.merge(rep)
    print(total.summary())
    assert total.within_budget
