"""Verification straight from hidden states (tensor-core product with the softmax partials in its
epilogue) against the CPU oracle (needs a B200).

Two bars.  (1) The call's logits are the binary32 accumulations the tensor cores deliver; the same
values can be written out (fef_lmhead_logits), and on those values the call must equal the oracle
at the standard bar: integers exact outside the 1e-6 margins, confidences to 1e-5.  (2) Against
the oracle's double-precision product of the same bfloat16 bytes the logits differ by the
accumulation error of d binary32 additions, about 2^-24 sqrt(d) sum|h_k w_k| (checked element by
element), which moves confidences by up to a few 1e-5 relative and decisions whose margin is
below that; there the bar is: integers exact outside margins of 1e-3, confidences to 2e-4."""
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import lmhead as olm
from oracle.compare import ParityReport, compare_verify

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fef():
    import paper_2605_14305_b200 as lib

    lib.load(build_if_missing=True)
    return lib


def _hidden_case(B, K, V, d, seed, noise=0.35):
    """Draft hidden states ~ N(0, 1), target = draft + N(0, noise^2), weight ~ N(0, 4 / d): logits of
    standard deviation 2 whose two versions differ by about N(0, (2 noise)^2), as in the logit-level workloads."""
    g = torch.Generator(device="cuda").manual_seed(seed)
    Hq = torch.randn((B * K, d), generator=g, device="cuda")
    Hp = Hq + noise * torch.randn((B * K, d), generator=g, device="cuda")
    W = torch.randn((V, d), generator=g, device="cuda") * (2.0 / math.sqrt(d))
    Hq, Hp, W = Hq.to(torch.bfloat16), Hp.to(torch.bfloat16), W.to(torch.bfloat16)
    lq = (Hq.float() @ W.float().T)
    u = torch.rand(lq.shape, generator=g, device="cuda").clamp_(1e-12, 1 - 1e-7)
    tok = torch.argmax(lq - torch.log(-torch.log(u)), dim=-1).to(torch.int32).view(B, K)
    return Hq, Hp, W, tok


@pytest.mark.parametrize("rows,V,d", [(128, 256, 64), (100, 300, 72), (77, 4097, 264), (300, 5000, 1024),
                                      (32, 126464, 256), (64, 4096, 4096)])
def test_logits_are_the_product_to_binary32_accumulation_error(fef, rows, V, d):
    g = torch.Generator(device="cuda").manual_seed(rows + V + d)
    H = torch.randn((rows, d), generator=g, device="cuda").to(torch.bfloat16)
    W = (torch.randn((V, d), generator=g, device="cuda") * (2.0 / math.sqrt(d))).to(torch.bfloat16)
    out, st = fef.fef_lmhead_logits(H, W)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    ref = olm.lmhead_logits(H.cpu(), W.cpu())
    scale = olm.lmhead_logits(H.cpu().abs(), W.cpu().abs())          # sum_k |h_k w_k| per element
    err = np.abs(out[:, :V].cpu().numpy().astype(np.float64) - ref)
    bound = 4.0 * 2.0 ** -24 * math.sqrt(d) * scale + 1e-30
    assert (err <= bound).all(), (float(err.max()), float((err / bound).max()))
    # twice the same call: the same bits (no race between the epilogue and the next tile's products)
    again, _ = fef.fef_lmhead_logits(H, W)
    torch.cuda.synchronize()
    assert torch.equal(out[:, :V], again[:, :V])


CASES = [
    # B, K, V, d, T
    (2, 4, 256, 64, 1.0),
    (3, 5, 1000, 128, 0.8),
    (10, 16, 5000, 512, 1.0),       # 160 rows: two row tiles per matrix; V not a multiple of the column tile
    (4, 8, 4099, 256, 1.0),         # V not a multiple of four
    (4, 8, 4096, 256, 1.0),
    (4, 8, 4096, 4096, 0.7),
    (4, 8, 126464, 256, 1.0),
    (2, 8, 126464, 4096, 1.0),
]


@pytest.mark.parametrize("B,K,V,d,T", CASES)
def test_verification_from_hidden_states(fef, B, K, V, d, T):
    Hq, Hp, W, tok = _hidden_case(B, K, V, d, seed=B * 1000 + V + d)
    row_len = None
    if B >= 3:
        row_len = torch.tensor([K, 0, max(K - 3, 1)] + [K] * (B - 3), dtype=torch.int32, device="cuda")
    r = fef.fef_lmhead_verify(Hq, Hp, W, tok, T, 21, 6, row_len=row_len)
    torch.cuda.synchronize()
    assert int(r.device_status.item()) == 0
    ga, gt, gc = r.accept_len.cpu().numpy(), r.tokens.cpu().numpy(), r.conf.cpu().numpy()

    # (1) on the binary32 logits the call itself sees: the standard bar
    lq, _ = fef.fef_lmhead_logits(Hq, W)
    lp, _ = fef.fef_lmhead_logits(Hp, W)
    torch.cuda.synchronize()
    ldo = lq.shape[1]
    ref32 = oracle.spec_verify(lq.view(B, K, ldo).cpu(), lp.view(B, K, ldo).cpu(), tok.cpu(), T, 21, 6,
                               row_len=None if row_len is None else row_len.cpu(), V=V)
    assert ref32["status"] == 0
    rep = compare_verify(ga, gt, gc, ref32)
    assert rep.ok, rep.mismatches[:5]
    assert rep.within_budget

    # (2) against the double-precision product of the same bytes: the wider bar
    ref64 = olm.lmhead_spec_verify(Hq.cpu(), Hp.cpu(), W.cpu(), tok.cpu(), B, K, T, 21, 6,
                                   row_len=None if row_len is None else row_len.cpu())
    wide = compare_verify(ga, gt, gc, ref64, margin=1e-3, conf_rtol=2e-4)
    assert wide.ok, wide.mismatches[:5]
    print(rep.summary(), "| against the float64 product:", wide.summary())
    assert (ga[ga >= 0] < K).any() or B * K < 16      # the residual path ran


def test_two_calls_in_a_row_and_argument_errors(fef):
    B, K, V, d = 3, 6, 3000, 128
    Hq, Hp, W, tok = _hidden_case(B, K, V, d, seed=5)
    ws = torch.empty(fef.fef_lmhead_verify_workspace_bytes(B, K, V, d), dtype=torch.uint8, device="cuda")
    a = fef.fef_lmhead_verify(Hq, Hp, W, tok, 1.0, 3, 1, workspace=ws)
    a = tuple(x.clone() for x in a)
    b = fef.fef_lmhead_verify(Hq, Hp, W, tok, 1.0, 3, 1, workspace=ws)
    torch.cuda.synchronize()
    assert all(torch.equal(x, y) for x, y in zip(a, b))
    with pytest.raises(fef.FefError):
        fef.fef_lmhead_verify(Hq, Hp, W, tok, 0.0, 3, 1)                      # sampling mode only
    with pytest.raises(fef.FefError):
        fef.fef_lmhead_verify(Hq, Hp, W, tok, 1.0, 3, 1, workspace=ws[:1024])  # scratch too small
    with pytest.raises(fef.FefError):
        fef.fef_lmhead_verify(Hq[:, :100].contiguous(), Hp, W, tok, 1.0, 3, 1)
    bad = tok.clone()
    bad[1, 2] = V
    r = fef.fef_lmhead_verify(Hq, Hp, W, bad, 1.0, 3, 1)
    torch.cuda.synchronize()
    assert int(r.device_status.item()) == fef.FEF_ERR_TOKEN_RANGE and int(r.accept_len[1].item()) == -1
    assert int(r.accept_len[0].item()) == int(a[0][0].item())
