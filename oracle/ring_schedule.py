"""Ring-schedule simulator for the paper's Algo. 1-3 -- TEST INFRASTRUCTURE ONLY (documentation value).

The paper schedules the scalar operations of self-attention onto a unidirectional ring of m synchronous
processing engines (PEs): in every cycle each PE does one multiply (or exponential, or division), one
accumulation and one transfer to its right neighbour (Sec. 2.1).  Its three algorithms are index formulas that
say, for every cycle and PE, which partial sum w'_AB the PE holds and which vector component C it multiplies.

The GPU library does not use these schedules (a tensor core issues 128 x 128 x 16 products, not scalars); this
module rebuilds them for tiny n so that the claims the paper makes about them can be checked mechanically:

  * coverage     every multiply-accumulate the scheme needs is issued exactly once, nothing else is;
  * ring rule    a partial sum that is "transferred to the adjacent PE" is the one its right neighbour works
                 on in the next cycle;
  * cycle count  cycles per phase, to compare with the #Cycles columns of Tables I and II.

Conventions of the listings: indices are 1-based, % is the non-negative remainder, \\ is integer division,
d = n (Sec. 3.2), m divides n.  Everything here is plain Python over small integers.
"""
from __future__ import annotations

from collections import Counter


def _groups(n):
    """Number of packed groups minus one: h' of Algo. 2 and Algo. 3."""
    return (n - 1) // 2 if n % 2 else n // 2 - 1


def _component(l, j, i, n, m):
    """Vector component C the PE l multiplies in step j of block i (the same formula in all three listings)."""
    return (l + ((j - 1) // m) * m + (i - 1) * m - 1) % n + 1


def _home(l, j, i, m):
    """Row index (l - j) % m + (i - 1) m + 1: which of the block's m partial sums PE l holds in step j."""
    return (l - j) % m + (i - 1) * m + 1


# ------------------------------------------------------------------------------------------------ phase 1 schedules
def phase1_algo1(n, m):
    """Algo. 1, phase 1: for every row h of the weight matrix, n/m blocks of n steps.  Returns a list of cycles;
    a cycle is a list over the m PEs of (A, B, C), the multiply-accumulate w'_AB += q_A[C] k_B[C]."""
    cycles = []
    for h in range(1, n + 1):
        for i in range(1, n // m + 1):
            for j in range(1, n + 1):
                row = []
                for l in range(1, m + 1):
                    B = (_home(l, j, i, m) - 2) % n + 1          # ((l-j)%m + (i-1)m - 1) % n + 1
                    row.append((h, B, _component(l, j, i, n, m)))
                cycles.append(row)
    return cycles


def phase1_algo2(n, m):
    """Algo. 2, phase 1 (query = key = value): groups of n weights taken along cyclic diagonals (Sec. 4.2); group h
    holds the weights w'_AB with A = B +- h (mod n).  Returns (compute cycles as above, reuse-transfer cycles of
    the listing read literally = sum of p' over the groups with (h % m) > 1, times n/m blocks)."""
    cycles, transfers = [], 0
    hp = _groups(n)
    offsets = list(range(0, hp + 1)) + ([n // 2] if n % 2 == 0 else [])      # even n: the whole n/2-th diagonal too
    for idx, h in enumerate(offsets):
        extra_group = n % 2 == 0 and idx == len(offsets) - 1
        for i in range(1, n // m + 1):
            for j in range(1, n + 1):
                row = []
                for l in range(1, m + 1):
                    B = (_home(l, j, i, m) - 2) % n + 1
                    if extra_group:
                        A = (B + n // 2 - 1) % n + 1
                    elif (h % m) <= m / 2:
                        A = (B + h - 1) % n + 1
                    else:
                        A = (B - h - 1) % n + 1
                    row.append((A, B, _component(l, j, i, n, m)))
                cycles.append(row)
            if not extra_group and (h % m) > 1:
                transfers += (h % m) if (h % m) <= m / 2 else m - (h % m)
    return cycles, transfers


def reuse_transfer_cycles_minus_one(n, m):
    """The other reading of the reuse transfers: p' - 1 cycles per block (the last hop coincides with the store)."""
    t = 0
    for h in range(0, _groups(n) + 1):
        if (h % m) > 1:
            p = (h % m) if (h % m) <= m / 2 else m - (h % m)
            t += (p - 1) * (n // m)
    return t


def phase1_algo3(n, m):
    """Algo. 3, phase 1 (masked): row n - h is packed with row h into a group of n weights (Sec. 5.2); for even n
    the middle row n/2 forms a half-used group of its own.  Returns cycles; an idle PE slot is None."""
    cycles = []
    hp = _groups(n)
    for h in range(0, hp + 1):
        for i in range(1, n // m + 1):
            for j in range(1, n + 1):
                row = []
                for l in range(1, m + 1):
                    A, B = n - h, _home(l, j, i, m)
                    if A < B:
                        A, B = h, B % (n - h)
                        if B == 0:
                            B = n - h              # (B is 1-based: the remainder 0 stands for the last of the n - h)
                    row.append((A, B, _component(l, j, i, n, m)) if 1 <= B <= A and A >= 1 else None)
                cycles.append(row)
    if n % 2 == 0:
        for i in range(1, n // m + 1):
            for j in range(1, n + 1):
                row = []
                for l in range(1, m + 1):
                    A, B = n // 2, _home(l, j, i, m)
                    row.append((A, B, _component(l, j, i, n, m)) if A >= B else None)
                cycles.append(row)
    return cycles


# ------------------------------------------------------------------------------------------------ checks
def coverage(cycles):
    """Counter of the (A, B, C) triples issued (idle slots ignored)."""
    c = Counter()
    for row in cycles:
        for op in row:
            if op is not None:
                c[op] += 1
    return c


def ring_rule_violations(cycles, n):
    """Counts hand-overs that break the ring: within a block of n steps the partial sum (A, B) that PE l works on in
    step j must be the one PE l + 1 (cyclically) works on in step j + 1.  Blocks are consecutive runs of n cycles."""
    bad = 0
    m = len(cycles[0])
    for start in range(0, len(cycles), n):
        block = cycles[start:start + n]
        for j in range(len(block) - 1):
            for l in range(m):
                a, b = block[j][l], block[j + 1][(l + 1) % m]
                if a is None or b is None:
                    if a is not b and not (a is None or b is None):
                        bad += 1
                    continue
                if a[:2] != b[:2]:
                    bad += 1
    return bad


def needed_pairs(n, scheme):
    """(A, B) pairs the scheme computes in phase 1 (element level, the paper's selection for the symmetric scheme)."""
    if scheme == "full":
        return {(a, b) for a in range(1, n + 1) for b in range(1, n + 1)}
    if scheme == "masked":
        return {(a, b) for a in range(1, n + 1) for b in range(1, a + 1)}
    pairs = set()
    hp = _groups(n)
    for b in range(1, n + 1):
        for off in list(range(0, hp + 1)) + ([n // 2] if n % 2 == 0 else []):
            pairs.add(((b + off - 1) % n + 1, b))
    return pairs


def total_cycles(n, m, algo):
    """#Cycles of the whole computation: phase 1 as scheduled here, phase 2 (exponent-accumulate step and division step:
    n/m blocks of n steps each) and phase 3 (the loops of phase 1 again; for Algo. 2 those of Algo. 1).  For Algo. 2
    the reuse transfers are returned separately, in both readings: (cycles without them, literal, minus-one)."""
    phase2 = 2 * (n // m) * n
    if algo == 1:
        p1 = len(phase1_algo1(n, m))
        return p1 + phase2 + p1
    if algo == 3:
        p1 = len(phase1_algo3(n, m))
        return p1 + phase2 + p1
    cyc, literal = phase1_algo2(n, m)
    base = len(cyc) + phase2 + len(phase1_algo1(n, m))
    return base, literal, reuse_transfer_cycles_minus_one(n, m)
