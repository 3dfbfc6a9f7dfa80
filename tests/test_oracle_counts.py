"""Pins for the oracle's operation census: numbers the paper prints, and its closed forms.

Nothing here asks the oracle what to expect: expectations come from tests/golden/*.txt (values
printed in the paper's Tables I and II and Sec. 6) and from the formulas of Sec. 3.2, 4.2, 5.2
typed here independently.
"""
import os

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append(line.split())
    return out


def _census(n, d, scheme, selection=oracle.SEL_MINIMAL, seed=0):
    rng = np.random.default_rng(seed)
    Q, K, V = (rng.standard_normal((n, d)) for _ in range(3))
    _, c, _, _ = oracle.attention_slice(Q, K, V, scheme, 1.0, selection)
    return c


TABLE1 = _rows("table1_cycles.txt")
TABLE2 = _rows("table2_cycles.txt")


@pytest.mark.parametrize("row", TABLE1 + [r[:3] for r in TABLE2])
def test_full_census_equals_table_algo1_cycles_times_pes(row):
    # Tables I, II, column "Algo.1": every PE does one operation per cycle, d = n.
    n, m, algo1 = int(row[0]), int(row[1]), int(row[2])
    c = _census(n, n, oracle.FULL)
    assert c.total == algo1 * m
    assert (c.mac1, c.eac, c.div, c.mac3) == (n * n * n, n * n, n * n, n * n * n)


@pytest.mark.parametrize("row", [r for r in TABLE2 if not r[4].endswith("x")])
def test_masked_census_equals_table2_ideal_times_pes(row):
    # Table II, parenthesised / asterisked values = (#computations)/(#PEs) of the masked scheme.
    n, m, ideal = int(row[0]), int(row[1]), int(row[4])
    c = _census(n, n, oracle.MASKED)
    assert c.total == ideal * m


@pytest.mark.parametrize("row", [r for r in TABLE1 if (int(r[0]), int(r[1])) in ((3, 3), (4, 4))])
def test_symmetric_census_equals_table1_algo2_cycles_times_pes(row):
    # Table I, column "Algo.2", the two rows whose schedules need no extra reuse-transfer cycles
    # ((h % m) > 1 never holds): cycles * m is then the number of operations, even-n trade-off included.
    n, m, algo2 = int(row[0]), int(row[1]), int(row[4])
    c = _census(n, n, oracle.SYMMETRIC, oracle.SEL_PAPER)
    assert c.total == algo2 * m


@pytest.mark.parametrize("n,d", [(1, 1), (2, 5), (7, 3), (16, 4), (33, 8), (64, 64), (96, 17)])
def test_closed_forms_of_the_text(n, d):
    full = _census(n, d, oracle.FULL)
    assert full.as_dict() == dict(mac1=d * n * n, eac=n * n, div=n * n, mac3=d * n * n)      # Sec. 3.2
    assert full.total == 2 * d * n * n + 2 * n * n                                             # Sec. 4.2
    kept = n * (n + 1) // 2
    masked = _census(n, d, oracle.MASKED)
    assert masked.as_dict() == dict(mac1=d * kept, eac=kept, div=kept, mac3=d * kept)        # Sec. 5.1, 5.2
    sym_p = _census(n, d, oracle.SYMMETRIC, oracle.SEL_PAPER)
    want = d * n * (n + 1) // 2 if n % 2 else d * n * (n + 2) // 2                              # Sec. 4.2
    assert sym_p.as_dict() == dict(mac1=want, eac=n * n, div=n * n, mac3=d * n * n)
    sym_m = _census(n, d, oracle.SYMMETRIC, oracle.SEL_MINIMAL)
    assert sym_m.mac1 == d * n * (n + 1) // 2                                                   # Sec. 4.1
    assert (sym_m.eac, sym_m.div, sym_m.mac3) == (n * n, n * n, d * n * n)


def test_reductions_are_near_25_and_50_percent():
    # Abstract / Sec. 4.2 / Sec. 5.2: "near 25%" and "near 50%" of the original computations.
    n = d = 192
    full = _census(n, d, oracle.FULL).total
    sym = _census(n, d, oracle.SYMMETRIC, oracle.SEL_PAPER).total
    msk = _census(n, d, oracle.MASKED).total
    assert 0.24 < 1 - sym / full < 0.25
    assert 0.49 < 1 - msk / full < 0.50


def test_algo3_cycle_model_reproduces_table2_and_sec6_example():
    # Sec. 5.2: rows are packed in pairs (i, n-i) so each of the G groups fills n slots; phases 1 and 3
    # take G*n*n/m cycles each (d = n), phase 2 takes 2*n*n/m.  This checks the fixture against the
    # paper's own formula, and that the slots cover the oracle's masked census.
    def cycles(n, m):
        G = (n + 1) // 2 if n % 2 else n // 2 + 1
        return 2 * G * n * n // m + 2 * n * n // m, G
    for r in TABLE2:
        n, m, algo3 = int(r[0]), int(r[1]), int(r[5])
        cyc, G = cycles(n, m)
        assert cyc == algo3
        assert G * n >= _census(n, n, oracle.MASKED).eac > (G - 1) * n
    with open(os.path.join(GOLD, "closed_forms.txt")) as f:
        val = [float(l.split()[1]) for l in f if l.startswith("algo3_cycles_n10000")][0]
    n, m = 10000, 5000
    assert cycles(n, m)[0] == n * n * (n + 2) // m + 2 * n * n // m
    assert round(cycles(n, m)[0] / 1e6, 2) == val


@pytest.mark.parametrize("scheme,sel", [(oracle.FULL, 0), (oracle.MASKED, 0), (oracle.SYMMETRIC, 0),
                                        (oracle.SYMMETRIC, 1)])
@pytest.mark.parametrize("n,d", [(5, 3), (12, 4), (31, 2)])
def test_tile_census_with_unit_tiles_is_the_element_census(scheme, sel, n, d):
    t = oracle.tile_counts(n, d, scheme, 1, 1, sel)
    c = _census(n, d, scheme, sel)
    assert (t.issued_mac1, t.issued_mac3) == (c.mac1, c.mac3)
    assert (t.useful_mac1, t.useful_mac3) == (c.mac1, c.mac3)


@pytest.mark.parametrize("n", [128, 256, 512, 1024, 1152])
def test_tile_census_closed_forms_at_128x128(n):
    d, b = 64, 128
    T = n // b
    full = oracle.tile_counts(n, d, oracle.FULL, b, b)
    assert (full.tiles1, full.tiles3) == (T * T, T * T)
    assert full.issued_mac1 == d * n * n == full.useful_mac1
    msk = oracle.tile_counts(n, d, oracle.MASKED, b, b)
    assert (msk.tiles1, msk.tiles3) == (T * (T + 1) // 2,) * 2
    assert msk.issued_mac1 == T * (T + 1) // 2 * b * b * d
    assert msk.useful_mac1 == d * n * (n + 1) // 2
    sym = oracle.tile_counts(n, d, oracle.SYMMETRIC, b, b)
    assert (sym.tiles1, sym.tiles3) == (T * (T + 1) // 2, T * T)
    assert sym.useful_mac1 == d * n * (n + 1) // 2 and sym.useful_mac3 == d * n * n


def test_tile_census_clips_ragged_tiles():
    t = oracle.tile_counts(200, 8, oracle.MASKED, 128, 128)
    # tiles (0,0) 128x128, (1,0) 72x128, (1,1) 72x72 are issued; (0,1) holds nothing needed
    assert t.tiles1 == 3
    assert t.issued_mac1 == 8 * (128 * 128 + 72 * 128 + 72 * 72)
