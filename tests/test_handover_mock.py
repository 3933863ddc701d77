"""The workspace hand-over protocol of the decode kernels, run by CPU threads (tests/handover_mock.cpp).

Slots hold 0xFFFFFFFF while empty and their one reader empties them again; T entries carry the call
number taken from the departure counter; every poll is bounded.  The cases below run the protocol
over many calls on one workspace, and make a bounded wait expire by withholding one writer: the
status word gets the time-out bit, every CTA still leaves, the departure counter still advances,
and after the reset the interface asks for the next call is clean.  Nothing here touches a GPU."""
import os
import re
import subprocess

import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
TIMEOUT_BIT = 1 << 7
LINE = re.compile(r"call (\d+) status (\d+) departures (\d+) wrong (\d+) left (\d+)")


@pytest.fixture(scope="module")
def mock(tmp_path_factory):
    exe = str(tmp_path_factory.mktemp("mock") / "handover_mock")
    subprocess.run(["g++", "-O2", "-std=c++17", "-pthread", os.path.join(HERE, "handover_mock.cpp"), "-o", exe], check=True)
    return exe


def run(exe, n_ctas, n_units, calls, withhold, poll_limit):
    out = subprocess.run([exe, str(n_ctas), str(n_units), str(calls), str(withhold), str(poll_limit)],
                         check=True, capture_output=True, text=True, timeout=120).stdout.splitlines()
    rows = [tuple(int(x) for x in LINE.match(l).groups()) for l in out if l.startswith("call")]
    return rows, out


@pytest.mark.parametrize("n_ctas,n_units", [(1, 5), (4, 4), (6, 37), (8, 3)])
def test_many_calls_share_one_workspace(mock, n_ctas, n_units):
    rows, _ = run(mock, n_ctas, n_units, 25, 0, 1 << 26)
    assert len(rows) == 25
    for k, (call, status, departures, wrong, left) in enumerate(rows, 1):
        assert call == k and status == 0
        assert departures == k * n_ctas           # every CTA left, once per call
        assert wrong == 0                         # every fetched entry was this call's sum, added in list order
        assert left == 0                          # the readers emptied every slot


def test_a_wait_that_runs_out_sets_the_status_and_nobody_stays_behind(mock):
    n_ctas, n_units = 5, 11
    rows, out = run(mock, n_ctas, n_units, 6, 3, 2000)
    assert len(rows) == 6
    for call, status, departures, wrong, left in rows[:2]:
        assert status == 0 and wrong == 0 and left == 0 and departures == call * n_ctas
    call, status, departures, wrong, left = rows[2]
    assert status & TIMEOUT_BIT                   # the bounded poll gave up
    assert (status >> 16) & 64                    # ... and says it was waiting for partials of T
    assert departures == 3 * n_ctas               # the call still ended: every CTA left
    assert wrong > 0                              # its result is not to be used
    assert out[out.index(f"call 3 status {status} departures {departures} wrong {wrong} left {left}") + 1] == "reset"
    for k, (call, status, departures, wrong, left) in enumerate(rows[3:], 1):
        assert status == 0 and wrong == 0 and left == 0
        assert departures == k * n_ctas           # counted from the reset
