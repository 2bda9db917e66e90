"""The five benchmark configurations at their full extent against the CPU oracle (needs a B200).

Config 0 (tiny, 100 denoising steps) is in test_gpu_parity.py.  Here: config 1 as stated (8 blocks
of 32 positions, 8 denoising steps each, every call checked), config 2 (all windows, three noise
levels, and the mean committed length against Theorem 2), config 3 and the benchmark's workload
(all 64 windows, both temperatures), config 4 (all 18 sweep points; every call at B = 1, the
first, the half-way and the last round of each denoising step at B >= 8, all windows)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import loop as oloop
from oracle.compare import ParityReport, compare_verify
from paper_2605_14305_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fef():
    import paper_2605_14305_b200 as lib

    lib.load(build_if_missing=True)
    return lib


def _verify_both(fef, q, p, tok, T, seed, step, row_len=None, draft_log2_norm=None):
    r = fef.fef_spec_verify(q, p, tok, T, seed, step, row_len=row_len, draft_log2_norm=draft_log2_norm)
    torch.cuda.synchronize()
    assert int(r.device_status.item()) == 0
    ga, gt, gc = r.accept_len.cpu().numpy(), r.tokens.cpu().numpy(), r.conf.cpu().numpy()
    ref = oracle.spec_verify(q.cpu(), p.cpu(), tok.cpu(), T, seed, step,
                             row_len=None if row_len is None else row_len.cpu())
    assert ref["status"] == 0
    rep = compare_verify(ga, gt, gc, ref)
    assert rep.ok, rep.mismatches[:5]
    return rep, (ga, gt, gc)


def _theorem2(q, p, T, row_len=None):
    """Per window the mean and variance of the committed count C (accepted drafts plus the corrected
    position) from Theorem 2's argument with per-position acceptance probabilities
    alpha_i = sum_x min{pi_i, rho_i} taken from the oracle: P(C >= l + 1) = prod_{i < l} alpha_i."""
    q, p = q.cpu(), p.cpu()
    B, K, _ = q.shape
    mean, var = np.zeros(B), np.zeros(B)
    for b in range(B):
        n = K if row_len is None else int(row_len[b])
        if n == 0:
            continue
        alpha = np.array([oracle.row_laws(p[b, i], q[b, i], T)[3] for i in range(n)])
        reach = np.concatenate([[1.0], np.cumprod(alpha[:-1])])
        mean[b] = reach.sum()
        var[b] = ((2 * np.arange(n) + 1) * reach).sum() - mean[b] ** 2
    return mean, var


def _select_both(fef, conf, mask, k):
    pos, cnt = fef.fef_remask_select(conf, mask, k)
    opos, ocnt = oracle.remask_select(conf.cpu(), mask.cpu(), k)
    assert (pos.cpu().numpy() == opos).all() and (cnt.cpu().numpy() == ocnt).all()
    return opos, ocnt


# ------------------------------------------------------------------ config 1 ----
def test_config1_llada_single_stream_as_stated(fef):
    """B = 1, generation length 256 = 8 blocks of K = 32, V = 126464, bf16, T = 1, 8 denoising steps
    per block, re-mask k = 8: every verification call and every selection checked."""
    from paper_2605_14305_b200.decode_loop import run_decode_loop

    w = synth.LLADA_SINGLE
    total = ParityReport()
    rounds = 0
    for block in range(w.gen_len // w.K):
        def logits_fn(rnd, window, row_len):
            return synth.make_logits(w, seed=2000 + rnd, device="cuda")

        def draft_fn(q, rnd):
            return synth.sample_draft_tokens(q, w.temperature, 6000 + rnd)

        def verify_fn(q, p, tok, rl, rnd):
            rep, got = _verify_both(fef, q, p, tok, w.temperature, 11, rnd, row_len=rl)
            total.merge(rep)
            return got

        out = run_decode_loop(w.B, w.K, w.K, 8, w.remask_k, logits_fn, draft_fn, verify_fn,
                              lambda conf, mask, k: _select_both(fef, conf, mask, k), first_round=rounds)
        assert (out["tokens"] >= 0).all()
        assert sum(out["committed_per_round"]) == w.K + 7 * w.remask_k
        rounds += out["rounds"]
    print(total.summary(), "calls", rounds)
    assert total.windows == rounds and total.within_budget


# ------------------------------------------------------------------ config 2 ----
@pytest.mark.parametrize("sigma", [0.2, 0.7, 1.5])
def test_config2_llada_batched_sigma_sweep(fef, sigma):
    """B = 16, K = 32, V = 126464, bf16, T = 0.7: all windows against the oracle; then the mean
    committed length over many calls (fresh drafts and acceptance draws each) against Theorem 2."""
    w = synth.LLADA_BATCHED
    q, p, tok = synth.make_call(w, seed=int(sigma * 100), device="cuda", noise_std=sigma)
    rep, (ga, gt, gc) = _verify_both(fef, q, p, tok, w.temperature, 3, int(sigma * 10))
    assert rep.within_budget
    mask = torch.as_tensor(gc >= 0).to(torch.uint8).cuda()
    _select_both(fef, torch.as_tensor(gc).cuda(), mask, w.remask_k)

    mean, var = _theorem2(q, p, w.temperature)
    reps = 60
    committed = np.zeros(w.B)
    for s in range(reps):
        d = fef.fef_draft_sample(q, w.temperature, 1234, 100 + s)
        r = fef.fef_spec_verify(q, p, d.tokens, w.temperature, 1234, 100 + s, draft_log2_norm=d.log2_norm)
        committed += np.minimum(r.accept_len.cpu().numpy() + 1, w.K)
    observed = committed.sum() / (reps * w.B)
    expected = mean.mean()
    se = np.sqrt(var.sum() / reps) / w.B
    alpha = 1.0 - 1.0 / max(expected, 1.0)   # the alpha a constant-rate window of this mean would have (large K)
    print("sigma", sigma, rep.summary(), "committed per window: observed %.4f, Theorem 2 %.4f +- %.4f (alpha ~ %.3f)"
          % (observed, expected, se, alpha))
    assert abs(observed - expected) < 4.5 * se


# ------------------------------------------------- config 3 and the benchmark ----
@pytest.mark.parametrize("T", [1.0, 0.0])
def test_config3_dream_large_batch_all_windows(fef, T):
    """B = 64, K = 32, V = 152064, bf16, Zipf-biased logits, in the launch configuration the
    benchmark uses: all 64 windows."""
    w = synth.DREAM_LARGE.with_(temperature=T)
    q, p, tok = synth.make_call(w, seed=33, device="cuda")
    if T == 0.0:  # most drafts equal the arg-max so that windows get past position 0
        top = p.float().argmax(-1).to(torch.int32)
        tok = torch.where(torch.rand(tok.shape, device="cuda") < 0.15, tok, top)
    rep, (ga, gt, gc) = _verify_both(fef, q, p, tok, T, 17, 4)
    assert rep.windows == 64 and rep.within_budget
    print(rep.summary(), "mean accept_len", ga.mean())


def test_headline_workload_all_windows_and_theorem2(fef):
    """The benchmark's workload (B = 64, K = 32, V = 126464, bf16, T = 1): all windows; mean committed
    length over many calls against Theorem 2 on the first 8 windows."""
    w = synth.HEADLINE
    q, p, tok = synth.make_call(w, seed=5, device="cuda")
    rep, (ga, _, _) = _verify_both(fef, q, p, tok, w.temperature, 99, 1)
    assert rep.windows == 64 and rep.within_budget
    nb = 8
    mean, var = _theorem2(q[:nb], p[:nb], w.temperature)
    reps = 100
    committed = np.zeros(nb)
    for s in range(reps):
        d = fef.fef_draft_sample(q, w.temperature, 4321, 500 + s)
        r = fef.fef_spec_verify(q, p, d.tokens, w.temperature, 4321, 500 + s)
        committed += np.minimum(r.accept_len[:nb].cpu().numpy() + 1, w.K)
    observed, expected = committed.sum() / (reps * nb), mean.mean()
    se = np.sqrt(var.sum() / reps) / nb
    print(rep.summary(), "committed per window: observed %.4f, Theorem 2 %.4f +- %.4f" % (observed, expected, se))
    assert abs(observed - expected) < 4.5 * se


# ------------------------------------------------------------------ config 4 ----
SWEEP = [(B, K, dt) for dt in (torch.bfloat16, torch.float32) for B in (1, 8, 64) for K in (8, 32, 64)]


@pytest.mark.parametrize("B,K,dtype", SWEEP, ids=["B%d-K%d-%s" % (B, K, "bf16" if dt == torch.bfloat16 else "f32")
                                                  for B, K, dt in SWEEP])
def test_config4_long_generation_sweep_point(fef, B, K, dtype):
    """Generation length 1024, V = 126464, target = draft + N(0, 0.7^2), logits drawn anew on the
    device every round, the full loop (window, draft draws, verification, commit; LowConf and
    re-masking between the two denoising steps) on the device-resident state until nothing is
    masked.  The oracle re-does the draft draws, the verification and the bookkeeping of the checked
    rounds on the device's inputs.  Sampling rule: B = 1 every round; B >= 8 the first round, the
    first round after which at least half of the positions are resolved, and the last round of each
    denoising step; all windows of a checked round.  Beside it: committed positions of the checked
    rounds against Theorem 2's expectation for the same logits."""
    from paper_2605_14305_b200.decode_loop import run_decode_loop_device

    w = synth.HEADLINE.with_(B=B, K=K, dtype=dtype, noise_std=0.7)
    L, T, seed = 1024, w.temperature, 77
    reuse_norm = (K != 32)            # both forms of the verification call appear in the sweep
    total = ParityReport()
    st = dict(checked=0, half=False, committed=0.0, expected=0.0, var=0.0, remasks=0)

    def logits_fn(rnd, window, row_len, inputs):
        return synth.make_logits(w, seed=7000 + rnd, device="cuda")

    def on_round(rnd, d):
        if rnd is None:               # re-masking: LowConf on the device's state against the oracle
            tok_b, conf_b, in_b = (x.cpu().numpy() for x in d["before"])
            opos, ocnt = oracle.remask_select(conf_b, in_b, 8)
            assert (d["positions"].cpu().numpy() == opos).all() and (d["count"].cpu().numpy() == ocnt).all()
            oloop.remask(tok_b, conf_b, in_b, opos, ocnt)
            assert (d["tokens"].cpu().numpy() == tok_b).all() and (d["in_step"].cpu().numpy() == in_b).all()
            st["remasks"] += 1
            st["half"] = True         # the second step is short: only its first and last rounds matter
            st["first_of_step"] = True
            return
        left = int((d["tokens"] == oloop.MASK).sum().item())
        first = rnd == 0 or st.pop("first_of_step", False)
        half = not st["half"] and left <= B * L // 2
        if half:
            st["half"] = True
        if not (B == 1 or first or half or left == 0):
            return
        tok_b, conf_b, in_b = (x.cpu().numpy() for x in d["before"])
        ow, orl, oun = oloop.next_window(tok_b, K)
        assert (d["window"].cpu().numpy() == ow).all() and (d["row_len"].cpu().numpy() == orl).all()
        od = oracle.draft_sample(d["q"].cpu(), T, seed, rnd, row_len=orl)
        used = np.arange(K)[None, :] < orl[:, None]
        dt = d["draft"].tokens.cpu().numpy()
        sure = od["gumbel_gap"] > 1e-6
        assert (dt[used & sure] == od["tokens"][used & sure]).all()
        r = d["result"]
        ga, gt, gc = r.accept_len.cpu().numpy(), r.tokens.cpu().numpy(), r.conf.cpu().numpy()
        ref = oracle.spec_verify(d["q"].cpu(), d["p"].cpu(), dt, T, seed, rnd, row_len=orl)
        rep = compare_verify(ga, gt, gc, ref)
        assert rep.ok, rep.mismatches[:5]
        total.merge(rep)
        on = oloop.commit(tok_b, conf_b, in_b, ow, orl, ga, gt, gc)
        assert (d["committed"].cpu().numpy() == on).all()
        assert (d["tokens"].cpu().numpy() == tok_b).all() and (d["conf"].cpu().numpy() == conf_b).all()
        assert (d["in_step"].cpu().numpy() == in_b).all()
        if st["checked"] < 3 or B == 1 and st["checked"] % 16 == 0:   # Theorem 2 beside a few of them
            nb = min(B, 4)
            mean, var = _theorem2(d["q"][:nb], d["p"][:nb], T, row_len=orl[:nb])
            st["expected"] += mean.sum()
            st["var"] += var.sum()
            st["committed"] += float(on[:nb].sum())
        st["checked"] += 1

    out = run_decode_loop_device(fef, B, L, K, 2, 8, logits_fn, T, seed, on_round=on_round,
                                 reuse_draft_norm=reuse_norm)
    assert (out["tokens"] >= 0).all()
    assert sum(out["committed_per_round"]) == B * L + B * 8 and st["remasks"] == 1
    assert st["checked"] >= (out["rounds"] if B == 1 else 4)
    z = (st["committed"] - st["expected"]) / max(np.sqrt(st["var"]), 1e-9)
    print(total.summary(), "rounds", out["rounds"], "checked", st["checked"],
          "committed in the Theorem-2 sample: %.0f, expected %.1f (z = %.2f)" % (st["committed"], st["expected"], z))
    assert total.within_budget and abs(z) < 4.5
