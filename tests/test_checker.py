"""The parity checker itself (oracle/compare.py), on hand-made disagreements: every kind of wrong
answer must be reported, and only differences inside the stated margins may be excused."""
import numpy as np

from oracle.compare import CONF_RTOL, MARGIN, ParityReport, compare_verify


def _ref(B=3, K=4):
    """A reference result: window 0 accepts everything, window 1 rejects at 2, window 2 at 0."""
    accept_len = np.array([K, 2, 0], dtype=np.int32)[:B]
    tokens = np.full((B, K), -1, dtype=np.int32)
    conf = np.full((B, K), -1.0)
    margin = np.full((B, K), np.inf)
    gap = np.full(B, np.inf)
    rng = np.random.default_rng(1)
    for b in range(B):
        n = min(accept_len[b] + 1, K)
        tokens[b, :n] = rng.integers(0, 1000, n)
        conf[b, :n] = rng.uniform(0.01, 0.9, n)
        margin[b, :min(accept_len[b] + 1, K)] = 0.25      # every test made, far from the boundary
        if accept_len[b] < K:
            gap[b] = 0.5
    return dict(status=0, accept_len=accept_len, tokens=tokens, conf=conf, accept_margin=margin, gumbel_gap=gap)


def _got(ref):
    return ref["accept_len"].copy(), ref["tokens"].copy(), ref["conf"].astype(np.float32).copy()


def test_identical_results_pass_and_count_draws():
    ref = _ref()
    rep = compare_verify(*_got(ref), ref, ledger=False)
    assert rep.ok and rep.excused == 0 and rep.windows == 3
    assert rep.draws == 4 + 3 + 1 + 2          # acceptance tests made + residual draws
    assert rep.max_conf_rel_err < 1e-7


def test_wrong_accepted_token_is_a_mismatch():
    ref = _ref()
    a, t, c = _got(ref)
    t[0, 1] += 1
    assert not compare_verify(a, t, c, ref, ledger=False).ok


def test_wrong_corrected_token_at_a_wide_gap_is_a_mismatch_and_inside_the_gap_an_excuse():
    ref = _ref()
    a, t, c = _got(ref)
    t[1, 2] += 1
    rep = compare_verify(a, t, c, ref, ledger=False)
    assert not rep.ok and rep.excused == 0
    ref["gumbel_gap"][1] = 0.5 * MARGIN
    rep = compare_verify(a, t, c, ref, ledger=False)
    assert rep.ok and rep.excused == 1
    ref["gumbel_gap"][1] = 2.0 * MARGIN
    assert not compare_verify(a, t, c, ref, ledger=False).ok


def test_accept_len_off_by_one_either_way_is_a_mismatch_at_a_wide_margin():
    for delta in (-1, +1):
        ref = _ref()
        a, t, c = _got(ref)
        a[1] += delta
        rep = compare_verify(a, t, c, ref, ledger=False)
        assert not rep.ok and rep.excused == 0, delta


def test_accept_len_difference_is_excused_only_when_the_deciding_draw_is_inside_the_margin():
    ref = _ref()
    a, t, c = _got(ref)
    a[1] = 3                                      # the implementation accepted position 2 as well
    ref["accept_margin"][1, 2] = 0.5 * MARGIN
    rep = compare_verify(a, t, c, ref, ledger=False)
    assert rep.ok and rep.excused == 1 and rep.near_margin == 1
    ref["accept_margin"][1, 2] = 1.5 * MARGIN
    assert not compare_verify(a, t, c, ref, ledger=False).ok
    # a near-margin draw somewhere else does not excuse a difference at a clear one
    ref["accept_margin"][1, 2] = 0.25
    ref["accept_margin"][1, 0] = 0.5 * MARGIN
    assert not compare_verify(a, t, c, ref, ledger=False).ok


def test_confidence_off_by_two_tolerances_is_a_mismatch_and_by_half_a_tolerance_is_not():
    ref = _ref()
    a, t, c = _got(ref)
    c64 = ref["conf"].copy()
    c64[0, 2] *= 1.0 + 2.0 * CONF_RTOL
    assert not compare_verify(a, t, c64, ref, ledger=False).ok
    c64 = ref["conf"].copy()
    c64[0, 2] *= 1.0 - 0.5 * CONF_RTOL
    rep = compare_verify(a, t, c64, ref, ledger=False)
    assert rep.ok and 0.4 * CONF_RTOL < rep.max_conf_rel_err < 0.6 * CONF_RTOL
    # the corrected token's confidence is checked too
    c64 = ref["conf"].copy()
    c64[1, 2] *= 1.0 + 2.0 * CONF_RTOL
    assert not compare_verify(a, t, c64, ref, ledger=False).ok


def test_tail_beyond_the_committed_prefix_must_hold_the_sentinels():
    ref = _ref()
    a, t, c = _got(ref)
    c[1, 3] = 0.5                                 # a confidence where nothing was committed
    assert not compare_verify(a, t, c, ref, ledger=False).ok
    a, t, c = _got(ref)
    t[2, 2] = 17                                  # a token where nothing was committed
    assert not compare_verify(a, t, c, ref, ledger=False).ok


def test_error_windows_must_agree():
    ref = _ref()
    ref["accept_len"][2] = -1
    ref["tokens"][2] = -1
    ref["conf"][2] = -1.0
    a, t, c = _got(ref)
    assert compare_verify(a, t, c, ref, ledger=False).ok
    a[2] = 0
    assert not compare_verify(a, t, c, ref, ledger=False).ok
    a, t, c = _got(ref)
    ref2 = _ref()
    a2, t2, c2 = _got(ref2)
    a2[0] = -1                                    # an error reported where the oracle has none
    assert not compare_verify(a2, t2, c2, ref2, ledger=False).ok


def test_tiny_confidences_are_held_to_the_binary32_grid_not_beyond():
    ref = _ref()
    ref["conf"][0, 0] = 3.0e-42                   # subnormal in binary32
    a, t, c = _got(ref)                            # rounds to the nearest subnormal: allowed
    assert compare_verify(a, t, c, ref, ledger=False).ok
    c[0, 0] = np.float32(6.0e-42)                  # twice the value: not a rounding difference
    assert not compare_verify(a, t, c, ref, ledger=False).ok
    ref["conf"][0, 1] = 1.0e-30                   # small but normal: the relative bar applies
    a, t, c = _got(ref)
    c64 = c.astype(np.float64)
    c64[0, 1] = 1.0e-30 * (1 + 3e-5)
    assert not compare_verify(a, t, c64, ref, ledger=False).ok


def test_reports_merge():
    ref = _ref()
    a, t, c = _got(ref)
    total = ParityReport()
    total.merge(compare_verify(a, t, c, ref, ledger=False))
    t[0, 0] += 1
    total.merge(compare_verify(a, t, c, ref, ledger=False))
    assert total.windows == 6 and len(total.mismatches) == 1 and not total.ok


def test_excuse_budget_rule():
    r = ParityReport(draws=5000, excused=1)
    assert not r.within_budget                      # one in 5000 is far above 1e-5
    r = ParityReport(draws=5000, excused=0)
    assert r.within_budget
    r = ParityReport(draws=400000, excused=3)
    assert r.within_budget
    r = ParityReport(draws=400000, excused=4)
    assert not r.within_budget
