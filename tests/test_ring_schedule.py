"""The paper's ring schedules (Algo. 1-3) rebuilt from their index formulas for the (n, m) of Tables I and II:
every multiply-accumulate the scheme needs is issued exactly once, partial sums move only to the right neighbour,
and the cycle counts are the tables' (tests/golden/table1_cycles.txt, table2_cycles.txt).  For Algo. 2 the table
also contains reuse-transfer cycles, which no single reading of the listing reproduces in all rows: the test states
which rows each reading matches."""
import os
from collections import Counter

import pytest

from oracle import ring_schedule as rs

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _table(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                rows.append(line.split())
    return rows


TABLE1 = [(int(r[0]), int(r[1]), int(r[2]), int(r[4])) for r in _table("table1_cycles.txt")]           # n m algo1 algo2
TABLE2 = [(int(r[0]), int(r[1]), int(r[2]), int(r[5])) for r in _table("table2_cycles.txt")]           # n m algo1 algo3
SIZES = sorted({(r[0], r[1]) for r in TABLE1 + TABLE2} | {(8, 4), (12, 4), (9, 3)})


@pytest.mark.parametrize("n,m", SIZES)
def test_algo1_issues_every_product_once_and_obeys_the_ring(n, m):
    cyc = rs.phase1_algo1(n, m)
    cov = rs.coverage(cyc)
    assert set(cov.values()) == {1}
    assert set(cov) == {(a, b, c) for a in range(1, n + 1) for b in range(1, n + 1) for c in range(1, n + 1)}
    assert rs.ring_rule_violations(cyc, n) == 0
    assert all(op is not None for row in cyc for op in row)          # every PE busy in every cycle (Sec. 3.2)
    assert len(cyc) * m == n ** 3                                    # d n^2 multiply-accumulates with d = n


@pytest.mark.parametrize("n,m", SIZES)
def test_algo3_issues_exactly_the_unmasked_products(n, m):
    cyc = rs.phase1_algo3(n, m)
    cov = rs.coverage(cyc)
    assert set(cov.values()) == {1}
    assert set(cov) == {(a, b, c) for (a, b) in rs.needed_pairs(n, "masked") for c in range(1, n + 1)}
    assert sum(cov.values()) == n * n * (n + 1) // 2                 # Sec. 5.2: d n(n+1)/2 with d = n
    assert rs.ring_rule_violations(cyc, n) == 0
    # odd n: rows n-h and h fill every slot; even n: the middle row's group is half used
    idle = sum(op is None for row in cyc for op in row)
    assert idle == (0 if n % 2 else n * n // 2)


@pytest.mark.parametrize("n,m", SIZES)
def test_algo2_issues_one_member_of_each_symmetric_pair(n, m):
    cyc, _ = rs.phase1_algo2(n, m)
    got = Counter()
    for (a, b, c), k in rs.coverage(cyc).items():
        got[(min(a, b), max(a, b), c)] += k
    want = Counter()
    for a in range(1, n + 1):
        for b in range(a, n + 1):
            # the unordered pair at cyclic distance n/2 (even n) is issued twice: the balance trade-off of Sec. 4.2 item 4
            twice = n % 2 == 0 and b - a == n // 2
            for c in range(1, n + 1):
                want[(a, b, c)] = 2 if twice else 1
    assert got == want
    assert sum(got.values()) == (n * n * (n + 1) // 2 if n % 2 else n * n * (n + 2) // 2)      # Sec. 4.2 counts, d = n
    assert rs.ring_rule_violations(cyc, n) == 0


@pytest.mark.parametrize("n,m,algo1,algo2", TABLE1)
def test_table1_cycle_counts(n, m, algo1, algo2):
    assert rs.total_cycles(n, m, 1) == algo1
    base, literal, minus_one = rs.total_cycles(n, m, 2)
    implied = algo2 - base                       # reuse-transfer cycles the table's Algo. 2 entry contains
    assert implied >= 0
    # neither reading of "for p in [1, p']: transfer" gives the table's column in every row
    matches_literal = implied == literal
    matches_minus_one = implied == minus_one
    expected = {(3, 3): (True, True), (4, 4): (True, True), (5, 5): (False, False), (6, 3): (True, False),
                (6, 6): (False, True), (15, 5): (False, True), (15, 15): (False, True)}
    assert (matches_literal, matches_minus_one) == expected[(n, m)]


@pytest.mark.parametrize("n,m,algo1,algo3", TABLE2)
def test_table2_cycle_counts(n, m, algo1, algo3):
    assert rs.total_cycles(n, m, 1) == algo1
    assert rs.total_cycles(n, m, 3) == algo3
