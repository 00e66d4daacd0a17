"""Halton-sequence broadcast and the SSP rule: oracle against the paper's worked example, library against the oracle."""
import math
import os

from oracle import sfb_schedule as sch
from paper_1511_08486_b200 import binding as B
from paper_1511_08486_b200.build import build_library

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "halton_p6_q2.txt")


def test_oracle_matches_the_papers_worked_example():
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    seen = 0
    for r in rows:
        if r[0] == "offsets":
            P, Q = int(r[1]), int(r[2])
            assert sch.halton_offsets(P, Q) == [int(x) for x in r[3:]]
            seen += 1
        else:
            P, Q, machine = int(r[0]), int(r[1]), int(r[2])
            # the paper numbers machines 1..P and applies (p + offset) % P to those numbers: 0 stands for machine P
            peers = sorted(x if x != 0 else P for x in sch.halton_peers(machine % P, P, Q))
            assert peers == [int(x) for x in r[3:]]
            seen += 1
    assert seen == 3
    # the sequence itself: 1/2, 1/4, 3/4, 1/8, 3/8, 5/8, 7/8
    assert sch.halton_fractions(7) == [(1, 2), (1, 4), (3, 4), (1, 8), (3, 8), (5, 8), (7, 8)]
    # with Q = P - 1 >= the number of distinct offsets on a power-of-two P, every other worker is reached
    assert sorted(sch.halton_peers(3, 8, 7)) == [0, 1, 2, 4, 5, 6, 7]


def test_ssp_rule_special_cases():
    assert sch.ssp_may_proceed(5, [5, 5, 5], 0)                # BSP: everyone caught up
    assert not sch.ssp_may_proceed(6, [5, 6, 6], 0)            # BSP: one worker behind -> wait
    assert sch.ssp_may_proceed(6, [5, 6, 6], 1) and not sch.ssp_may_proceed(8, [5, 8, 8], 2)
    assert sch.ssp_may_proceed(10 ** 9, [0, 0], math.inf)      # ASP never waits


def test_library_matches_oracle():
    build_library()
    for P in (1, 2, 6, 7, 12, 16, 100):
        for Q in (0, 1, 2, 4, 7):
            for p in (0, P // 2, P - 1):
                assert B.sfb_halton_peers(P, Q, p) == sch.halton_peers(p, P, Q)
    for t_p, tau, s in ((5, [5, 5], 0), (6, [5, 6], 0), (6, [5, 6], 1), (9, [5, 9, 2], 3), (9, [5, 9, 2], 7)):
        assert B.sfb_ssp_may_proceed(t_p, tau, s) == sch.ssp_may_proceed(t_p, tau, s)
    assert B.sfb_ssp_may_proceed(10 ** 12, [0, 1], -1) is True
