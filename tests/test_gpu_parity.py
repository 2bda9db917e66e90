"""CUDA library against the CPU oracle, element by element, through the C ABI (needs a B200)."""
import math

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


def _gpu_verify(fef, q, p, tok, T, seed, step, row_len=None, V=None):
    r = fef.fef_spec_verify(q, p, tok, T, seed, step, row_len=row_len, V=V)
    torch.cuda.synchronize()
    return (r.accept_len.cpu().numpy(), r.tokens.cpu().numpy(), r.conf.cpu().numpy(), int(r.device_status.item()))


def _check(fef, q, p, tok, T, seed, step, row_len=None, V=None, expect_status=0) -> ParityReport:
    """q, p, tok: CUDA tensors.  Runs both sides on the same bytes and compares."""
    ga, gt, gc, gs = _gpu_verify(fef, q, p, tok, T, seed, step, row_len, V)
    ref = oracle.spec_verify(q.cpu(), p.cpu(), tok.cpu(), T, seed, step,
                             row_len=None if row_len is None else row_len.cpu(), V=V)
    assert ref["status"] == expect_status
    assert gs == expect_status
    rep = compare_verify(ga, gt, gc, ref)
    assert rep.ok, rep.mismatches[:5]
    return rep


def _random_case(B, K, V, dtype, noise, seed, ld=None, scale=2.0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    ld = V if ld is None else ld
    q = torch.randn((B, K, ld), generator=g, device="cuda") * scale
    p = q + torch.randn((B, K, ld), generator=g, device="cuda") * noise
    q, p = q.to(dtype), p.to(dtype)
    if ld > V:  # padding must never be read
        q[:, :, V:] = float("nan")
        p[:, :, V:] = float("inf")
    tok = synth.sample_draft_tokens(q[:, :, :V].contiguous(), 1.0, seed + 1)
    return q, p, tok


SMALL_SHAPES = [
    # B, K, V, ld
    (1, 1, 1, 4), (2, 3, 3, 4), (3, 2, 4, 4), (2, 4, 7, 8), (5, 4, 8, 8), (2, 5, 9, 12), (3, 7, 33, 36),
    (4, 4, 1000, 1000), (1, 4, 1024, 1024), (2, 3, 4097, 4104), (7, 32, 260, 264), (2, 64, 520, 520),
    (300, 2, 64, 64), (2, 2, 40000, 40000), (1, 3, 70001, 70008),
    # short rows, many of them: the warp-per-row streaming kernel
    (40, 32, 1000, 1000), (100, 16, 4097, 4104), (1300, 1, 24, 24), (64, 32, 15808, 15808),
]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("T", [1.0, 0.7, 0.0])
def test_small_shapes_match_oracle(fef, dtype, T):
    total = ParityReport()
    for n, (B, K, V, ld) in enumerate(SMALL_SHAPES):
        if dtype == torch.bfloat16:
            ld = (ld + 7) // 8 * 8
        q, p, tok = _random_case(B, K, V, dtype, 0.8, 100 + n, ld=ld)
        if T == 0.0:  # make most drafts the arg-max so windows get past position 0
            top = p[:, :, :V].float().argmax(-1).to(torch.int32)
            keep = torch.rand(tok.shape, device="cuda") < 0.3
            tok = torch.where(keep, tok, top)
        total.merge(_check(fef, q, p, tok, T, seed=7 + n, step=n, V=V))
    print(total.summary())
    assert total.within_budget


def test_tiny_config_decode_loop_100_steps(fef):
    """Config 0: B=1, K=4, V=1024, fp32, T=1, re-mask k=2; every call checked against the oracle."""
    from paper_2605_14305_b200.decode_loop import run_decode_loop

    w = synth.TINY
    total = ParityReport()

    def logits_fn(rnd, window, row_len):
        return synth.make_logits(w, seed=1000 + rnd, device="cuda")

    def draft_fn(q, rnd):
        return synth.sample_draft_tokens(q, w.temperature, 5000 + rnd)

    def verify_fn(q, p, tok, rl, rnd):
        ga, gt, gc, gs = _gpu_verify(fef, q, p, tok, w.temperature, 0, rnd, row_len=rl)
        assert gs == 0
        ref = oracle.spec_verify(q.cpu(), p.cpu(), tok.cpu(), w.temperature, 0, rnd, row_len=rl.cpu())
        rep = compare_verify(ga, gt, gc, ref)
        assert rep.ok, rep.mismatches
        total.merge(rep)
        return ga, gt, gc

    def select_fn(conf, mask, k):
        pos, cnt = fef.fef_remask_select(conf, mask, k)
        opos, ocnt = oracle.remask_select(conf.cpu(), mask.cpu(), k)
        assert (pos.cpu().numpy() == opos).all() and (cnt.cpu().numpy() == ocnt).all()
        return opos, ocnt

    out = run_decode_loop(w.B, w.gen_len, w.K, 100, w.remask_k, logits_fn, draft_fn, verify_fn, select_fn)
    assert (out["tokens"] >= 0).all()
    assert out["rounds"] >= 100
    print(total.summary(), "rounds", out["rounds"])


def test_results_are_bit_identical_across_runs(fef):
    q, p, tok = _random_case(8, 16, 30000, torch.bfloat16, 0.9, 77)
    a = _gpu_verify(fef, q, p, tok, 0.9, 5, 6)
    for _ in range(3):
        b = _gpu_verify(fef, q, p, tok, 0.9, 5, 6)
        assert (a[0] == b[0]).all() and (a[1] == b[1]).all() and (a[2] == b[2]).all()


def test_identical_laws_accept_everything(fef):
    q, _, tok = _random_case(6, 32, 5000, torch.bfloat16, 0.5, 5)
    rep = _check(fef, q, q.clone(), tok, 0.8, 1, 1)
    ga, gt, _, _ = _gpu_verify(fef, q, q.clone(), tok, 0.8, 1, 1)
    assert (ga == 32).all() and (gt == tok.cpu().numpy()).all()


def test_row_len_and_empty_windows(fef):
    q, p, tok = _random_case(9, 8, 3000, torch.float32, 0.3, 9)
    row_len = torch.tensor([0, 1, 8, 3, 0, 8, 7, 2, 5], dtype=torch.int32, device="cuda")
    # garbage beyond row_len must not matter
    tok2 = tok.clone()
    for b in range(9):
        tok2[b, int(row_len[b]):] = -12345
        p[b, int(row_len[b]):] = float("nan")
    _check(fef, q, p, tok2, 1.0, 4, 4, row_len=row_len)


def test_minus_inf_and_zero_probability_conventions(fef):
    B, K, V = 4, 2, 64
    q, p, tok = _random_case(B, K, V, torch.float32, 0.5, 21)
    q[0, 0, 5] = -math.inf; tok[0, 0] = 5                         # rho(x)=0 < pi(x): accept
    q[1, 0, 6] = -math.inf; p[1, 0, 6] = -math.inf; tok[1, 0] = 6   # pi=rho=0: reject, residual draw
    p[2, 1, 10:40] = -math.inf                                     # masked vocabulary range
    q[3, 0] = p[3, 0]; p[3, 0, 9] = -math.inf; q[3, 0, 9] = -math.inf; tok[3, 0] = 9  # reject with zero residual
    rep = _check(fef, q, p, tok, 1.0, 8, 8)
    ga, gt, _, _ = _gpu_verify(fef, q, p, tok, 1.0, 8, 8)
    assert ga[0] >= 1 and ga[1] == 0 and ga[3] == 0
    assert gt[3, 0] == int(p[3, 0].argmax())


def test_data_errors_set_status_and_poison_only_their_window(fef):
    q, p, tok = _random_case(5, 4, 2000, torch.bfloat16, 0.5, 31)
    bad = p.clone(); bad[1, 2, 1234] = float("nan")
    _check(fef, q, bad, tok, 1.0, 1, 1, expect_status=7)
    bad = q.clone(); bad[2, 0, 0] = float("inf")
    _check(fef, bad, p, tok, 1.0, 1, 1, expect_status=7)
    bad = p.clone(); bad[4, 3, :] = -math.inf
    _check(fef, q, bad, tok, 1.0, 1, 1, expect_status=7)
    t2 = tok.clone(); t2[0, 1] = 2000
    _check(fef, q, p, t2, 1.0, 1, 1, expect_status=8)
    t2 = tok.clone(); t2[3, 0] = -1
    _check(fef, q, p, t2, 0.0, 1, 1, expect_status=8)
    # a later clean call resets the status word
    _check(fef, q, p, tok, 1.0, 1, 1, expect_status=0)


def test_far_apart_laws_reject_at_once_and_wide_dynamic_range(fef):
    g = torch.Generator(device="cuda").manual_seed(3)
    B, K, V = 3, 4, 9000
    q = torch.randn((B, K, V), generator=g, device="cuda") * 30.0      # logits spanning +-100
    p = torch.randn((B, K, V), generator=g, device="cuda") * 30.0
    tok = synth.sample_draft_tokens(q, 1.0, 4)
    _check(fef, q, p, tok, 1.0, 2, 2)
    _check(fef, q + 500.0, p - 500.0, tok, 1.0, 2, 3)                  # large common offsets
    # increasing ramp: the running reference has to move many times
    ramp = torch.linspace(-200, 200, V, device="cuda").expand(B, K, V).contiguous()
    _check(fef, ramp, (ramp * 0.98).contiguous(), tok, 1.0, 2, 4)


@pytest.mark.parametrize("B,L,k", [(1, 1, 1), (3, 17, 5), (8, 256, 8), (2, 1024, 2), (4, 33, 40), (2, 9, 0),
                                   (2, 8192, 8), (64, 1024, 8), (1, 5000, 5000), (3, 100, 32), (3, 100, 33), (2, 20, 32),
                                   (5, 2049, 31)])
def test_remask_select_matches_oracle(fef, B, L, k):
    g = torch.Generator(device="cuda").manual_seed(B * 1000 + L)
    conf = torch.rand((B, L), generator=g, device="cuda")
    conf[torch.rand((B, L), generator=g, device="cuda") < 0.3] = 0.25     # many exact ties
    conf[torch.rand((B, L), generator=g, device="cuda") < 0.05] = -1.0    # sentinels
    conf[torch.rand((B, L), generator=g, device="cuda") < 0.02] = 0.0
    conf[torch.rand((B, L), generator=g, device="cuda") < 0.02] = -0.0
    mask = (torch.rand((B, L), generator=g, device="cuda") < 0.6).to(torch.uint8)
    if B > 1:
        mask[1] = 0
    pos, cnt = fef.fef_remask_select(conf, mask, k)
    torch.cuda.synchronize()
    opos, ocnt = oracle.remask_select(conf.cpu(), mask.cpu(), k)
    assert (cnt.cpu().numpy() == ocnt).all()
    assert (pos.cpu().numpy() == opos).all()


def test_remask_select_nan_sorts_last(fef):
    conf = torch.tensor([[0.5, float("nan"), 0.1, float("inf"), float("nan"), -1.0]], device="cuda")
    mask = torch.ones_like(conf, dtype=torch.uint8)
    pos, cnt = fef.fef_remask_select(conf, mask, 6)
    opos, ocnt = oracle.remask_select(conf.cpu(), mask.cpu(), 6)
    assert pos.cpu().numpy().tolist() == opos.tolist() == [[5, 2, 0, 3, 1, 4]]


def test_host_buffer_entry_points_match_device_entry_points(fef):
    """fef_spec_verify_host / fef_remask_select_host: same results from pinned and from pageable host memory."""
    q, p, tok = _random_case(6, 8, 20000, torch.bfloat16, 0.7, 41)
    row_len = torch.tensor([8, 8, 3, 0, 8, 5], dtype=torch.int32, device="cuda")
    want = _gpu_verify(fef, q, p, tok, 0.9, 12, 13, row_len=row_len)
    arena = torch.empty(fef.fef_spec_verify_host_arena_bytes(6, 8, 20000, 20000, torch.bfloat16), dtype=torch.uint8,
                        device="cuda")
    for pin in (True, False):
        hq, hp, htok, hrl = (t.cpu().pin_memory() if pin else t.cpu() for t in (q, p, tok, row_len))
        got = fef.fef_spec_verify_host(hq, hp, htok, 0.9, 12, 13, arena, row_len=hrl)
        assert got.status == 0
        assert (got.accept_len.numpy() == want[0]).all() and (got.tokens.numpy() == want[1]).all()
        assert (got.conf.numpy() == want[2]).all()
    got = fef.fef_spec_verify_host(hq, hp, htok, 0.0, 12, 14, arena)
    want = _gpu_verify(fef, q, p, tok, 0.0, 12, 14)
    assert (got.tokens.numpy() == want[1]).all()
    conf = torch.rand(4, 300)
    mask = (torch.rand(4, 300) < 0.5).to(torch.uint8)
    arena2 = torch.empty(fef.fef_remask_select_host_arena_bytes(4, 300, 9), dtype=torch.uint8, device="cuda")
    pos, cnt = fef.fef_remask_select_host(conf, mask, 9, arena2)
    opos, ocnt = oracle.remask_select(conf, mask, 9)
    assert (pos.numpy() == opos).all() and (cnt.numpy() == ocnt).all()
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(fef.FefError) as err:
        fef.fef_spec_verify_host(hq, hp, htok, 0.9, 12, 13, small)
    assert err.value.status == fef.FEF_ERR_WORKSPACE


@pytest.mark.parametrize("B", [4, 32])
def test_profiled_entry_point_gives_identical_results_and_ordered_events(fef, B):
    # (the small call runs as one kernel unless timing marks are asked for: the row sums are then added
    # in another order, so its confidences agree to rounding, not to the bit)
    q, p, tok = _random_case(B, 16, 50000, torch.bfloat16, 0.7, 51)
    want = _gpu_verify(fef, q, p, tok, 1.0, 3, 3)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    for e in ev:
        e.record()
    r = fef.fef_spec_verify(q, p, tok, 1.0, 3, 3, stage_events=ev)
    torch.cuda.synchronize()
    assert (r.accept_len.cpu().numpy() == want[0]).all() and (r.tokens.cpu().numpy() == want[1]).all()
    if B == 32:
        assert (r.conf.cpu().numpy() == want[2]).all()
    else:
        np.testing.assert_allclose(r.conf.cpu().numpy(), want[2], rtol=2e-6)
    assert ev[0].elapsed_time(ev[1]) > 0 and ev[1].elapsed_time(ev[2]) > 0 and ev[2].elapsed_time(ev[3]) >= 0


def test_api_errors_with_real_buffers(fef):
    q, p, tok = _random_case(2, 4, 64, torch.float32, 0.5, 61)
    lib = fef.load()
    out = fef.fef_spec_verify(q, p, tok, 1.0, 0, 0)
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")

    def call(qq=q, V=64, ld=64, K=4, T=1.0, wsb=ws.numel(), wsp=None, dt=0):
        return lib.fef_spec_verify(qq.data_ptr(), p.data_ptr(), tok.data_ptr(), None, 2, K, V, ld, dt, T, 1, 1,
                                   out.accept_len.data_ptr(), out.tokens.data_ptr(), out.conf.data_ptr(),
                                   ws.data_ptr() if wsp is None else wsp, wsb, out.device_status.data_ptr(), None)
    assert call() == fef.FEF_OK
    assert call(wsb=16) == fef.FEF_ERR_WORKSPACE
    assert call(wsp=ws.data_ptr() + 8) == fef.FEF_ERR_WORKSPACE
    assert call(ld=32) == fef.FEF_ERR_INVALID_ARG
    assert call(K=65) == fef.FEF_ERR_INVALID_ARG
    assert call(T=-1.0) == fef.FEF_ERR_INVALID_ARG
    assert call(dt=5) == fef.FEF_ERR_DTYPE
    assert call(qq=q.view(-1)[1:]) == fef.FEF_ERR_ALIGNMENT
    assert call(V=10, ld=10) == fef.FEF_ERR_ALIGNMENT
    torch.cuda.synchronize()
    assert fef.fef_spec_verify_workspace_bytes(2, 4, 64, torch.float32) > 0
    assert fef.fef_spec_verify_workspace_bytes(2, 65, 64, torch.float32) == 0


# ------------------------------------------------------------ draft sampling ----
def _check_draft(fef, q, T, seed, step, row_len=None, V=None, expect_status=0):
    """fef_draft_sample against the oracle on the same bytes: tokens exact, except positions whose
    two best Gumbel scores lie within 1e-6 of each other (counted, must stay rare); normaliser to 1e-6."""
    r = fef.fef_draft_sample(q, T, seed, step, row_len=row_len, V=V)
    torch.cuda.synchronize()
    ref = oracle.draft_sample(q.cpu(), T, seed, step, row_len=None if row_len is None else row_len.cpu(), V=V)
    assert ref["status"] == expect_status and int(r.device_status.item()) == expect_status
    got = r.tokens.cpu().numpy()
    differ = got != ref["tokens"]
    excused = differ & (ref["gumbel_gap"] < 1e-6)
    assert not (differ & ~excused).any(), (np.argwhere(differ & ~excused)[:5], got[differ][:5], ref["tokens"][differ][:5])
    drawn = ref["tokens"] >= 0
    if drawn.any():
        Vv = q.shape[-1] if V is None else V
        Tn = T if T > 0 else 1.0
        want = torch.logsumexp(q.cpu()[..., :Vv].double() / float(np.float32(Tn)), dim=-1).numpy() / math.log(2.0)
        assert np.allclose(r.log2_norm.cpu().numpy()[drawn], want[drawn], rtol=0, atol=2e-5)
    return int(excused.sum()), int(drawn.sum())


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("T", [1.0, 0.7, 0.0])
def test_draft_sample_small_shapes_match_oracle(fef, dtype, T):
    excused = drawn = 0
    for n, (B, K, V, ld) in enumerate(SMALL_SHAPES):
        if dtype == torch.bfloat16:
            ld = (ld + 7) // 8 * 8
        q, _, _ = _random_case(B, K, V, dtype, 0.8, 300 + n, ld=ld)
        e, d = _check_draft(fef, q, T, seed=11 + n, step=n, V=V)
        excused += e
        drawn += d
    assert excused == 0 and drawn > 1000


def test_draft_sample_llada_and_dream_shapes_row_len_and_errors(fef):
    w = synth.LLADA_BATCHED.with_(B=4, K=8)
    q, _ = synth.make_logits(w, seed=5, device="cuda")
    assert _check_draft(fef, q, 0.7, 21, 1)[0] == 0
    rl = torch.tensor([8, 0, 3, 1], dtype=torch.int32, device="cuda")
    assert _check_draft(fef, q, 1.0, 21, 2, row_len=rl)[0] == 0
    wd = synth.DREAM_LARGE.with_(B=2, K=4)
    qd, _ = synth.make_logits(wd, seed=6, device="cuda")
    assert _check_draft(fef, qd, 1.0, 22, 3)[0] == 0
    assert _check_draft(fef, qd, 0.0, 22, 4)[0] == 0
    # one draw per row of a single window: the row is shared by many CTAs
    ws = synth.LLADA_SINGLE.with_(K=3)
    qs, _ = synth.make_logits(ws, seed=7, device="cuda")
    assert _check_draft(fef, qs, 1.0, 23, 5)[0] == 0
    # -inf entries are never drawn; NaN, +inf and a row without a finite logit are data errors
    qe = q.clone()
    qe[0, 0, ::2] = float("-inf")
    assert _check_draft(fef, qe, 1.0, 24, 6)[0] == 0
    qe[1, 2, 77] = float("nan")
    qe[2, 1, :] = float("-inf")
    qe[3, 0, 5] = float("inf")
    _check_draft(fef, qe, 1.0, 24, 7, expect_status=fef.FEF_ERR_NONFINITE)
    # the same call twice gives the same tokens (no race in the reductions)
    a = fef.fef_draft_sample(q, 0.9, 1, 1).tokens.clone()
    b = fef.fef_draft_sample(q, 0.9, 1, 1).tokens
    torch.cuda.synchronize()
    assert (a == b).all()


def test_draft_tokens_feed_verification(fef):
    """Drafts drawn on the device go straight into fef_spec_verify; the pair matches the oracle pair."""
    w = synth.LLADA_BATCHED.with_(B=3, K=16)
    q, p = synth.make_logits(w, seed=9, device="cuda")
    d = fef.fef_draft_sample(q, 0.7, 31, 4)
    _check(fef, q, p, d.tokens, 0.7, 31, 4)
    od = oracle.draft_sample(q.cpu(), 0.7, 31, 4)
    assert (d.tokens.cpu().numpy() == od["tokens"]).all()


def test_verification_with_the_draft_normalisers_streams_the_target_only(fef):
    """fef_draft_sample -> fef_spec_verify_with_draft_norm against the oracle pair, and against the plain call."""
    for w, T, seed in ((synth.LLADA_BATCHED.with_(B=5, K=16), 0.7, 41), (synth.LLADA_SINGLE.with_(K=8), 1.0, 42),
                       (synth.TINY.with_(B=90, K=32, V=3000, dtype=torch.bfloat16), 1.0, 44),  # short rows: warp per row
                       (synth.DREAM_LARGE.with_(B=3, K=8, dtype=torch.float32), 1.0, 43)):
        q, p = synth.make_logits(w, seed=seed, device="cuda")
        d = fef.fef_draft_sample(q, T, seed, 7)
        r = fef.fef_spec_verify(q, p, d.tokens, T, seed, 7, draft_log2_norm=d.log2_norm)
        plain = fef.fef_spec_verify(q, p, d.tokens, T, seed, 7)
        torch.cuda.synchronize()
        assert int(r.device_status.item()) == 0
        ref = oracle.spec_verify(q.cpu(), p.cpu(), d.tokens.cpu(), T, seed, 7)
        rep = compare_verify(r.accept_len.cpu().numpy(), r.tokens.cpu().numpy(), r.conf.cpu().numpy(), ref)
        assert rep.ok, rep.mismatches[:5]
        assert (r.accept_len == plain.accept_len).all() and (r.tokens == plain.tokens).all()
        assert torch.allclose(r.conf, plain.conf, rtol=1e-5, atol=0)
    # a bad normaliser poisons its window only
    bad = d.log2_norm.clone()
    bad[1, 0] = float("nan")
    r = fef.fef_spec_verify(q, p, d.tokens, T, seed, 7, draft_log2_norm=bad)
    torch.cuda.synchronize()
    assert int(r.device_status.item()) == fef.FEF_ERR_NONFINITE
    assert r.accept_len[1].item() == -1 and (r.accept_len[[0, 2]] == plain.accept_len[[0, 2]]).all()


def test_draft_draws_with_the_target_normalisers_and_verification_without_streaming(fef):
    """fef_draft_sample(target_logits=...) -> fef_spec_verify(draft_log2_norm=, target_log2_norm=):
    both tensors are read once, by the draft kernel; the pair equals the oracle pair and the plain calls."""
    total = ParityReport()
    for w, T, seed in ((synth.LLADA_BATCHED.with_(B=5, K=16), 0.7, 51), (synth.LLADA_SINGLE.with_(K=8), 1.0, 52),
                       (synth.TINY.with_(B=90, K=32, V=3001, dtype=torch.bfloat16), 1.0, 54),
                       (synth.TINY.with_(B=3, K=5, V=37), 1.0, 55),
                       (synth.DREAM_LARGE.with_(B=3, K=8, dtype=torch.float32), 1.0, 53)):
        q, p = synth.make_logits(w, seed=seed, device="cuda")
        if w.V % 8:  # rows must start on 16-byte boundaries: pad the pitch
            ld = (w.V + 7) // 8 * 8
            qq = torch.full((w.B, w.K, ld), float("nan"), dtype=q.dtype, device="cuda")
            pp = torch.full((w.B, w.K, ld), float("nan"), dtype=q.dtype, device="cuda")
            qq[:, :, :w.V], pp[:, :, :w.V] = q, p
            q, p = qq, pp
        rl = torch.randint(0, w.K + 1, (w.B,), dtype=torch.int32, device="cuda") if w.B > 2 else None
        d = fef.fef_draft_sample(q, T, seed, 7, row_len=rl, V=w.V, target_logits=p)
        plain_d = fef.fef_draft_sample(q, T, seed, 7, row_len=rl, V=w.V)
        r = fef.fef_spec_verify(q, p, d.tokens, T, seed, 7, row_len=rl, V=w.V, draft_log2_norm=d.log2_norm,
                                target_log2_norm=d.target_log2_norm)
        plain = fef.fef_spec_verify(q, p, d.tokens, T, seed, 7, row_len=rl, V=w.V)
        torch.cuda.synchronize()
        assert int(r.device_status.item()) == 0 and int(d.device_status.item()) == 0
        assert (d.tokens == plain_d.tokens).all() and (d.log2_norm == plain_d.log2_norm).all()
        n = np.full(w.B, w.K) if rl is None else rl.cpu().numpy()
        used = np.arange(w.K)[None, :] < n[:, None]
        want = torch.logsumexp(p.cpu()[..., :w.V].double() / float(np.float32(T)), dim=-1).numpy() / math.log(2.0)
        assert np.allclose(d.target_log2_norm.cpu().numpy()[used], want[used], rtol=0, atol=2e-5)
        assert (d.target_log2_norm.cpu().numpy()[~used] == 0).all()
        ref = oracle.spec_verify(q.cpu(), p.cpu(), d.tokens.cpu(), T, seed, 7, row_len=None if rl is None else rl.cpu(),
                                 V=w.V)
        rep = compare_verify(r.accept_len.cpu().numpy(), r.tokens.cpu().numpy(), r.conf.cpu().numpy(), ref)
        assert rep.ok, rep.mismatches[:5]
        total.merge(rep)
        assert (r.accept_len == plain.accept_len).all() and (r.tokens == plain.tokens).all()
        assert torch.allclose(r.conf, plain.conf, rtol=1e-5, atol=0)
    assert total.within_budget
    # a target row with bad data poisons its window only; temperature 0 ignores the normalisers
    pb = p.clone()
    pb[1, 0, 5] = float("nan")
    d2 = fef.fef_draft_sample(q, T, seed, 7, target_logits=pb)
    r2 = fef.fef_spec_verify(q, pb, d2.tokens, T, seed, 7, draft_log2_norm=d2.log2_norm, target_log2_norm=d2.target_log2_norm)
    g0 = fef.fef_spec_verify(q, p, d.tokens, 0.0, seed, 7, draft_log2_norm=d.log2_norm, target_log2_norm=d.target_log2_norm)
    g1 = fef.fef_spec_verify(q, p, d.tokens, 0.0, seed, 7)
    torch.cuda.synchronize()
    assert int(r2.device_status.item()) == fef.FEF_ERR_NONFINITE and int(r2.accept_len[1].item()) == -1
    assert (g0.tokens == g1.tokens).all() and (g0.conf == g1.conf).all()


def test_calls_on_a_stream_that_is_not_current_own_what_they_allocate(fef):
    """Outputs and scratch that the wrappers allocate belong to the stream the kernels run on: while
    calls are queued on a side stream, the current stream allocates and overwrites memory of the same
    sizes; every call still equals the oracle (draft draws and verification, large and small sizes)."""
    side = torch.cuda.Stream()
    for n, (B, K, V) in enumerate([(2, 8, 40000), (24, 32, 60000)]):
        q, p, tok = _random_case(B, K, V, torch.bfloat16, 0.7, 200 + n)
        ws_bytes = fef.fef_spec_verify_workspace_bytes(B, K, V, torch.bfloat16)
        side.wait_stream(torch.cuda.current_stream())
        results = []
        for step in range(6):
            d = fef.fef_draft_sample(q, 1.0, 9, step, stream=side)
            r = fef.fef_spec_verify(q, p, tok, 1.0, 9, step, stream=side)
            results.append((d, r))
            # the current stream takes and scribbles over blocks of the sizes the wrappers asked for
            for _ in range(4):
                torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device="cuda").fill_(0xAB)
                torch.empty((B, K), dtype=torch.int32, device="cuda").fill_(123456)
                torch.empty((B, K), dtype=torch.float32, device="cuda").fill_(7.0)
        torch.cuda.synchronize()
        for step, (d, r) in enumerate(results):
            ref = oracle.spec_verify(q.cpu(), p.cpu(), tok.cpu(), 1.0, 9, step)
            rep = compare_verify(r.accept_len.cpu().numpy(), r.tokens.cpu().numpy(), r.conf.cpu().numpy(), ref)
            assert rep.ok, rep.mismatches[:3]
            dref = oracle.draft_sample(q.cpu(), 1.0, 9, step)
            assert (d.tokens.cpu().numpy() == dref["tokens"]).all()
