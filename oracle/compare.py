"""Compare an implementation's verification outputs with the oracle's (test infrastructure).

The realisation is unique once the random stream is fixed, up to floating-point
margins: an acceptance draw whose |u - pi(x)/rho(x)| is below 1e-6, or a residual
draw whose two best Gumbel scores are closer than 1e-6, may legitimately come out
differently in binary32-accumulated arithmetic.  Such draws are counted as
ambiguous; everything else must match exactly (integers) or to 1e-5 relative
(confidences).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

MARGIN = 1e-6
CONF_RTOL = 1e-5
F32_SUBNORMAL_STEP = 2.0 ** -149   # spacing of binary32 numbers below 2^-126


@dataclass
class ParityReport:
    windows: int = 0
    draws: int = 0              # acceptance tests made + residual draws made (by the oracle)
    excused: int = 0            # windows that differ only through an ambiguous draw
    near_margin: int = 0        # draws within the margin, whether or not the results differ
    mismatches: list = field(default_factory=list)
    max_conf_rel_err: float = 0.0

    def merge(self, other: "ParityReport") -> "ParityReport":
        self.windows += other.windows
        self.draws += other.draws
        self.excused += other.excused
        self.near_margin += other.near_margin
        self.mismatches += other.mismatches
        self.max_conf_rel_err = max(self.max_conf_rel_err, other.max_conf_rel_err)
        return self

    @property
    def ok(self) -> bool:
        return not self.mismatches

    @property
    def within_budget(self) -> bool:
        """Excused windows must stay below 1e-5 of the draws made; with fewer than 1e5 draws that
        means none at all."""
        return self.excused == 0 if self.draws < 100000 else self.excused < 1e-5 * self.draws

    def summary(self) -> str:
        return ("windows=%d draws=%d near_margin=%d excused=%d mismatches=%d max_conf_rel_err=%.3g"
                % (self.windows, self.draws, self.near_margin, self.excused, len(self.mismatches),
                   self.max_conf_rel_err))


# Everything compared in this process, summed: a test session checks the excuse budget on it.
LEDGER = ParityReport()


def compare_verify(got_accept_len, got_tokens, got_conf, ref: dict, batch_offset: int = 0,
                   ledger: bool = True, margin: float = MARGIN, conf_rtol: float = CONF_RTOL) -> ParityReport:
    """``got_*``: arrays of the implementation under test for the same windows as ``ref``
    (the dict returned by ``oracle.spec_verify``).  The result is also added to ``LEDGER``
    unless ``ledger`` is false.  ``margin`` / ``conf_rtol``: other bars than the standard ones, for
    an implementation whose inputs themselves carry a stated error (logits from a binary32 product
    against the oracle's double-precision product); such comparisons stay out of the ledger."""
    rep = _compare_verify(got_accept_len, got_tokens, got_conf, ref, batch_offset, margin, conf_rtol)
    if margin != MARGIN or conf_rtol != CONF_RTOL:
        ledger = False
    if ledger:
        LEDGER.windows += rep.windows
        LEDGER.draws += rep.draws
        LEDGER.excused += rep.excused
        LEDGER.near_margin += rep.near_margin
        LEDGER.mismatches += rep.mismatches[:3]
        LEDGER.max_conf_rel_err = max(LEDGER.max_conf_rel_err, rep.max_conf_rel_err)
    return rep


def _compare_verify(got_accept_len, got_tokens, got_conf, ref: dict, batch_offset: int, MARGIN: float,
                    CONF_RTOL: float) -> ParityReport:
    ga = np.asarray(got_accept_len)
    gt = np.asarray(got_tokens)
    gc = np.asarray(got_conf, dtype=np.float64)
    ra, rt, rc = ref["accept_len"], ref["tokens"], ref["conf"]
    margin, gap = ref["accept_margin"], ref["gumbel_gap"]
    B, K = rt.shape
    rep = ParityReport(windows=B)
    rep.draws = int(np.isfinite(margin).sum() + np.isfinite(gap).sum())
    rep.near_margin = int((margin < MARGIN).sum() + (gap < MARGIN).sum())
    for b in range(B):
        tag = "window %d" % (b + batch_offset)
        if ra[b] < 0 or ga[b] < 0:
            if ra[b] != ga[b] or (gt[b] != rt[b]).any():
                rep.mismatches.append("%s: error window differs (got accept_len %d, oracle %d)" % (tag, ga[b], ra[b]))
            continue
        if ga[b] != ra[b]:
            i0 = min(ga[b], ra[b])
            if i0 < K and margin[b, i0] < MARGIN:
                rep.excused += 1
            else:
                rep.mismatches.append("%s: accept_len %d vs oracle %d (margin at %d = %.3g)"
                                      % (tag, ga[b], ra[b], i0, margin[b, min(i0, K - 1)]))
            continue
        a = ra[b]
        committed = rt[b] >= 0
        same = gt[b] == rt[b]
        if not same.all():
            only_at_a = a < K and same[np.arange(K) != a].all()
            if only_at_a and gap[b] < MARGIN:
                rep.excused += 1
                committed = committed & same
            else:
                rep.mismatches.append("%s: tokens %s vs oracle %s (gumbel gap %.3g)"
                                      % (tag, gt[b].tolist(), rt[b].tolist(), gap[b]))
                continue
        if (~committed & (gc[b] != -1.0) & same).any():
            rep.mismatches.append("%s: confidence beyond the committed prefix is not -1" % tag)
        if committed.any():
            r, g = rc[b][committed], gc[b][committed]
            denom = np.maximum(np.abs(r), 1e-300)
            rel = np.abs(g - r) / denom
            rel = np.where((r == 0) & (g == 0), 0.0, rel)
            # the confidences under test are binary32 numbers: a difference of at most one step of
            # the binary32 grid at that magnitude (a subnormal step for confidences below 2^-126) is
            # rounding of the output type, not of the method
            rel = np.where(np.abs(g - r) <= F32_SUBNORMAL_STEP, 0.0, rel)
            worst = float(rel.max())
            rep.max_conf_rel_err = max(rep.max_conf_rel_err, worst)
            if worst > CONF_RTOL:
                rep.mismatches.append("%s: confidence off by %.3g relative" % (tag, worst))
    return rep
