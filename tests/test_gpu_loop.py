"""Device-resident bookkeeping of the decoding loop (Algorithm 2) against the CPU oracle (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import loop as oloop
from oracle.compare import compare_verify
from paper_2605_14305_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fef():
    import paper_2605_14305_b200 as lib

    lib.load(build_if_missing=True)
    return lib


def _random_state(B, L, frac_masked, seed):
    rng = np.random.default_rng(seed)
    tokens = rng.integers(0, 50000, size=(B, L)).astype(np.int32)
    masked = rng.random((B, L)) < frac_masked
    if B > 1:
        masked[0] = False          # a finished row
        masked[-1] = True          # a row that is still all masked
    tokens[masked] = oloop.MASK
    conf = rng.random((B, L)).astype(np.float32)
    conf[masked] = -1.0
    in_step = ((rng.random((B, L)) < 0.5) & ~masked).astype(np.uint8)
    return tokens, conf, in_step


@pytest.mark.parametrize("B,L,K", [(1, 1, 1), (2, 5, 4), (3, 256, 32), (4, 257, 7), (5, 1000, 64), (2, 4097, 64),
                                   (64, 1024, 32), (1, 70000, 64)])
@pytest.mark.parametrize("frac", [0.0, 0.03, 0.5, 1.0])
def test_each_bookkeeping_call_matches_the_oracle(fef, B, L, K, frac):
    tokens, conf, in_step = _random_state(B, L, frac, seed=B * 1000 + L + K)
    rng = np.random.default_rng(L)
    d_tokens, d_conf, d_in = (torch.as_tensor(x).cuda() for x in (tokens, conf, in_step))

    # window
    w, rl, un = fef.fef_loop_next_window(d_tokens, K)
    ow, orl, oun = oloop.next_window(tokens, K)
    assert (w.cpu().numpy() == ow).all() and (rl.cpu().numpy() == orl).all() and (un.cpu().numpy() == oun).all()

    # verification inputs (kept small: B*K*L ints)
    draft = rng.integers(0, 50000, size=(B, K)).astype(np.int32)
    if B * K * L <= 1 << 24:
        x = fef.fef_loop_verification_inputs(d_tokens, w, rl, torch.as_tensor(draft).cuda())
        assert (x.cpu().numpy() == oloop.verification_inputs(tokens, ow, orl, draft)).all()

    # commit: every accept length 0 .. K, and one failed window
    accept = rng.integers(0, K + 1, size=B).astype(np.int32)
    accept = np.minimum(accept, orl)               # what verification can return for this window
    if B > 2:
        accept[1] = -1
    out_tok = rng.integers(0, 50000, size=(B, K)).astype(np.int32)
    out_conf = rng.random((B, K)).astype(np.float32)
    res = fef.VerifyResult(torch.as_tensor(accept).cuda(), torch.as_tensor(out_tok).cuda(),
                           torch.as_tensor(out_conf).cuda(), torch.zeros(1, dtype=torch.int32, device="cuda"))
    n = fef.fef_loop_commit(w, rl, res, d_tokens, d_conf, d_in)
    on = oloop.commit(tokens, conf, in_step, ow, orl, accept, out_tok, out_conf)
    assert (n.cpu().numpy() == on).all()
    assert (d_tokens.cpu().numpy() == tokens).all() and (d_conf.cpu().numpy() == conf).all()
    assert (d_in.cpu().numpy() == in_step).all()

    # re-masking of LowConf's choice
    for k in (0, 1, 8):
        if k > L or L > fef.FEF_MAX_REMASK_L:
            continue
        pos, cnt = fef.fef_remask_select(d_conf, d_in, k)
        opos, ocnt = oracle.remask_select(conf, in_step, k)
        assert (pos.cpu().numpy() == opos).all() and (cnt.cpu().numpy() == ocnt).all()
        fef.fef_loop_remask(pos, cnt, d_tokens, d_conf, d_in)
        oloop.remask(tokens, conf, in_step, opos, ocnt)
        assert (d_tokens.cpu().numpy() == tokens).all() and (d_conf.cpu().numpy() == conf).all()
        assert (d_in.cpu().numpy() == in_step).all()
        in_step[:] = (tokens != oloop.MASK) & (rng.random((B, L)) < 0.5)
        d_in.copy_(torch.as_tensor(in_step))


def test_bookkeeping_argument_errors(fef):
    t = torch.zeros((2, 8), dtype=torch.int32, device="cuda")
    with pytest.raises(fef.FefError):
        fef.fef_loop_next_window(t, 0)
    with pytest.raises(fef.FefError):
        fef.fef_loop_next_window(t, fef.FEF_MAX_K + 1)
    with pytest.raises(fef.FefError):
        fef.fef_loop_next_window(t.to(torch.int64), 4)
    with pytest.raises(fef.FefError):
        fef.fef_loop_next_window(t.cpu(), 4)


@pytest.mark.parametrize("B,K,L,dtype,T", [(1, 4, 64, torch.float32, 1.0), (3, 8, 100, torch.bfloat16, 1.0),
                                           (8, 32, 256, torch.bfloat16, 0.7), (2, 16, 96, torch.float32, 0.0)])
def test_device_resident_loop_matches_the_oracle_round_by_round(fef, B, K, L, dtype, T):
    """Three denoising steps with every call of every round re-done by the oracle on the device's
    inputs: window, draft draws, verification, commit, LowConf and re-masking; the oracle keeps
    its own copy of the state and the two must agree after every call."""
    from paper_2605_14305_b200.decode_loop import run_decode_loop_device

    w = synth.TINY.with_(B=B, K=K, V=2048, dtype=dtype, temperature=T, noise_std=0.6)
    st = dict(tokens=np.full((B, L), oloop.MASK, dtype=np.int32), conf=np.full((B, L), -1.0, dtype=np.float32),
              in_step=np.zeros((B, L), dtype=np.uint8), rounds=0, remasks=0)

    def logits_fn(rnd, window, row_len, inputs):
        return synth.make_logits(w, seed=300 + rnd, device="cuda")

    def on_round(rnd, d):
        if rnd is None:
            opos, ocnt = oracle.remask_select(st["conf"], st["in_step"], 5)
            assert (d["positions"].cpu().numpy() == opos).all() and (d["count"].cpu().numpy() == ocnt).all()
            oloop.remask(st["tokens"], st["conf"], st["in_step"], opos, ocnt)
            st["remasks"] += 1
        else:
            ow, orl, oun = oloop.next_window(st["tokens"], K)
            assert (d["window"].cpu().numpy() == ow).all() and (d["row_len"].cpu().numpy() == orl).all()
            assert (d["unresolved"].cpu().numpy() == oun).all()
            od = oracle.draft_sample(d["q"].cpu(), T, 11, rnd, row_len=orl)
            used = np.arange(K)[None, :] < orl[:, None]
            dt = d["draft"].tokens.cpu().numpy()
            assert (dt[used] == od["tokens"][used]).all()
            xin = oloop.verification_inputs(st["tokens"], ow, orl, dt)
            assert (d["inputs"].cpu().numpy() == xin).all()
            r = d["result"]
            ref = oracle.spec_verify(d["q"].cpu(), d["p"].cpu(), dt, T, 11, rnd, row_len=orl)
            ga, gt, gc = r.accept_len.cpu().numpy(), r.tokens.cpu().numpy(), r.conf.cpu().numpy()
            rep = compare_verify(ga, gt, gc, ref)
            assert rep.ok, rep.mismatches[:5]
            # the oracle's bookkeeping takes the device's verified values (they agree within the
            # floating-point tolerance above; the integer work after them must be exact)
            on = oloop.commit(st["tokens"], st["conf"], st["in_step"], ow, orl, ga, gt, gc)
            assert (d["committed"].cpu().numpy() == on).all()
            st["rounds"] += 1
        assert (d["tokens"].cpu().numpy() == st["tokens"]).all()
        assert (d["conf"].cpu().numpy() == st["conf"]).all()
        assert (d["in_step"].cpu().numpy() == st["in_step"]).all()

    out = run_decode_loop_device(fef, B, L, K, 3, 5, logits_fn, T, 11, on_round=on_round, build_inputs=True,
                                 reuse_draft_norm=(T > 0 and K % 16 == 0))
    assert (out["tokens"] >= 0).all()
    assert out["rounds"] == st["rounds"] and st["remasks"] == 2
    assert sum(out["committed_per_round"]) == B * L + 2 * B * 5


def test_at_round_entry_points_equal_the_plain_calls_at_the_summed_step(fef):
    """step + *device_round is the step: same draws, same verification, bit for bit."""
    w = synth.TINY.with_(B=3, K=8, V=4096, dtype=torch.bfloat16, noise_std=0.6)
    q, p = synth.make_logits(w, seed=5, device="cuda")
    rnd = torch.tensor([37], dtype=torch.int32, device="cuda")
    d0 = fef.fef_draft_sample(q, 1.0, 9, 100 + 37)
    d1 = fef.fef_draft_sample(q, 1.0, 9, 100, device_round=rnd)
    assert (d0.tokens == d1.tokens).all() and (d0.log2_norm == d1.log2_norm).all()
    for norm in (None, d0.log2_norm):
        r0 = fef.fef_spec_verify(q, p, d0.tokens, 1.0, 9, 137, draft_log2_norm=norm)
        r1 = fef.fef_spec_verify(q, p, d0.tokens, 1.0, 9, 100, draft_log2_norm=norm, device_round=rnd)
        assert (r0.accept_len == r1.accept_len).all() and (r0.tokens == r1.tokens).all() and (r0.conf == r1.conf).all()
    ref = oracle.spec_verify(q.cpu(), p.cpu(), d0.tokens.cpu(), 1.0, 9, 137)
    r1 = fef.fef_spec_verify(q, p, d0.tokens, 1.0, 9, 100, device_round=rnd)
    rep = compare_verify(r1.accept_len.cpu().numpy(), r1.tokens.cpu().numpy(), r1.conf.cpu().numpy(), ref)
    assert rep.ok, rep.mismatches[:5]
    # the counter moves only while some row has work left
    un = torch.tensor([0, 0, 0], dtype=torch.int32, device="cuda")
    fef.fef_loop_advance_round(rnd, un)
    assert int(rnd.item()) == 37
    un[1] = 2
    fef.fef_loop_advance_round(rnd, un)
    fef.fef_loop_advance_round(rnd)
    assert int(rnd.item()) == 39


@pytest.mark.parametrize("B,K,L,dtype,norm", [(2, 4, 40, torch.float32, False), (4, 8, 96, torch.bfloat16, True)])
def test_replayed_graph_of_a_round_equals_the_eager_device_loop(fef, B, K, L, dtype, norm):
    """One round captured as a CUDA graph and replayed (round number on the device) against the
    eager device-resident loop, which the test above checks against the oracle round by round."""
    from paper_2605_14305_b200.decode_loop import run_decode_loop_device, run_decode_loop_graph

    w = synth.TINY.with_(B=B, K=K, V=2048, dtype=dtype, noise_std=0.6)
    R = 16
    pool = [synth.make_logits(w, seed=900 + r, device="cuda") for r in range(R)]
    pool_q = torch.stack([x[0] for x in pool])
    pool_p = torch.stack([x[1] for x in pool])

    def eager_logits(rnd, window, row_len, inputs):
        return pool_q[rnd % R], pool_p[rnd % R]

    def graph_logits(device_round, window, row_len):
        idx = torch.remainder(device_round, R).to(torch.int64)
        return pool_q.index_select(0, idx)[0], pool_p.index_select(0, idx)[0]

    a = run_decode_loop_device(fef, B, L, K, 3, 4, eager_logits, 1.0, 21, reuse_draft_norm=norm)
    g = run_decode_loop_graph(fef, B, L, K, 3, 4, graph_logits, 1.0, 21, reuse_draft_norm=norm)
    torch.cuda.synchronize()
    assert g["rounds"] == a["rounds"]
    assert (g["tokens"] == a["tokens"]).all() and (g["conf"] == a["conf"]).all()
    assert (g["tokens"] >= 0).all()


def test_device_made_logits_are_seeded_shaped_and_reproducible(fef):
    B, K, V = 3, 5, 40000
    for dtype in (torch.bfloat16, torch.float32):
        q, p = fef.fef_synth_logits(B, K, V, dtype, 2.0, 0.7, seed=9, round=4, boost_fraction=0.01, boost=8.0)
        q2, p2 = fef.fef_synth_logits(B, K, V, dtype, 2.0, 0.7, seed=9, round=4, boost_fraction=0.01, boost=8.0)
        rnd = torch.tensor([3], dtype=torch.int32, device="cuda")
        q3, p3 = fef.fef_synth_logits(B, K, V, dtype, 2.0, 0.7, seed=9, round=1, boost_fraction=0.01, boost=8.0,
                                      device_round=rnd)
        q4, _ = fef.fef_synth_logits(B, K, V, dtype, 2.0, 0.7, seed=9, round=5, boost_fraction=0.01, boost=8.0)
        torch.cuda.synchronize()
        assert torch.equal(q, q2) and torch.equal(p, p2) and torch.equal(q, q3) and torch.equal(p, p3)
        assert not torch.equal(q, q4)
        qf, pf = q[:, :, :V].float(), p[:, :, :V].float()
        boosted = qf > 6.0                         # 2 sigma draws reach 6 with probability 1e-3; boosted ones start at 8 - 6
        assert abs(boosted.float().mean().item() - 5 / 512) < 2e-3
        base = torch.where(boosted, qf - 8.0, qf)
        assert abs(base.mean().item()) < 0.02 and abs(base.std().item() - 2.0) < 0.03
        d = pf - qf
        assert abs(d.mean().item()) < 0.01 and abs(d.std().item() - 0.7) < 0.02
        rows = qf.reshape(B * K, V)
        assert abs(torch.corrcoef(torch.stack([rows[0], rows[1]]))[0, 1].item()) < 0.02   # rows are independent


@pytest.mark.parametrize("B,K,L,dtype", [(1, 4, 40, torch.float32), (4, 8, 96, torch.bfloat16), (3, 32, 200, torch.bfloat16)])
def test_whole_loop_as_one_graph_launch_equals_the_eager_device_loop(fef, B, K, L, dtype):
    """fef_loop_run_synthetic (all rounds of all denoising steps as the body of a graph WHILE node, no host
    in between) against the eager device-resident loop making the same calls round by round."""
    from paper_2605_14305_b200.decode_loop import run_decode_loop_device

    V, T, seed, steps, k = 3000, 1.0, 33, 3, 4

    def logits_fn(rnd, window, row_len, inputs):
        return fef.fef_synth_logits(B, K, V, dtype, 2.0, 0.7, seed, rnd, boost_fraction=0.01, boost=8.0)

    a = run_decode_loop_device(fef, B, L, K, steps, k, logits_fn, T, seed, reuse_target_norm=True, V=V)
    g = fef.fef_loop_run_synthetic(B, L, K, V, dtype, T, seed, steps, k, 2.0, 0.7, boost_fraction=0.01, boost=8.0)
    torch.cuda.synchronize()
    assert g["device_status"] == 0
    assert g["rounds"] == a["rounds"]
    assert (g["tokens"] == a["tokens"]).all() and (g["conf"] == a["conf"]).all()
    assert (g["tokens"] >= 0).all()


def test_eager_loop_with_both_normalisers_matches_the_oracle_round_by_round(fef):
    """The calls the one-launch loop makes (device-made logits, draft draws that also reduce the target
    rows, verification that takes both normalisers), checked against the oracle on every round."""
    from paper_2605_14305_b200.decode_loop import run_decode_loop_device

    B, K, L, V, T, seed = 3, 8, 64, 5000, 0.9, 17
    st = dict(rounds=0)

    def logits_fn(rnd, window, row_len, inputs):
        return fef.fef_synth_logits(B, K, V, torch.bfloat16, 2.0, 0.7, seed, rnd, boost_fraction=0.01, boost=8.0)

    def on_round(rnd, d):
        if rnd is None:
            return
        orl = d["row_len"].cpu().numpy()
        od = oracle.draft_sample(d["q"].cpu(), T, seed, rnd, row_len=orl, V=V)
        used = np.arange(K)[None, :] < orl[:, None]
        dt = d["draft"].tokens.cpu().numpy()
        assert (dt[used] == od["tokens"][used]).all()
        ref = oracle.spec_verify(d["q"].cpu(), d["p"].cpu(), dt, T, seed, rnd, row_len=orl, V=V)
        r = d["result"]
        rep = compare_verify(r.accept_len.cpu().numpy(), r.tokens.cpu().numpy(), r.conf.cpu().numpy(), ref)
        assert rep.ok, rep.mismatches[:5]
        st["rounds"] += 1

    out = run_decode_loop_device(fef, B, L, K, 2, 3, logits_fn, T, seed, on_round=on_round, reuse_target_norm=True, V=V)
    assert (out["tokens"] >= 0).all() and st["rounds"] == out["rounds"]
