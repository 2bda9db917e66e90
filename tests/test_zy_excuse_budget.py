"""Whole-session excuse budget (needs a B200; collected after every other parity test).

A draw whose acceptance margin |u - pi/rho| or whose two best Gumbel scores lie within 1e-6 may come
out differently in binary32-accumulated arithmetic; windows that differ only through such a draw are
excused by the checker.  Over everything this session compared, the excused windows must stay below
1e-5 of the draws made (none at all while fewer than 1e5 draws were made), and nothing may be a
plain mismatch."""
import pytest

from oracle import compare

pytestmark = pytest.mark.gpu


def test_excused_windows_stay_below_one_in_1e5_draws():
    led = compare.LEDGER
    print("session:", led.summary())
    assert not led.mismatches, led.mismatches[:5]
    assert led.within_budget
